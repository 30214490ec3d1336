"""Device-memory bookkeeping for one quantised layer: owns the buffers that
qbp_layer_fwd / qbp_layer_bwd need (codes, parameters, saved statistics,
gradient copies, workspace) as torch tensors and passes their addresses
through the C ABI.  No arithmetic happens here."""
from __future__ import annotations

import torch

from . import binding as B


class QuantizedLayer:
    """conv: a binding.ConvDesc for a convolution layer (x NHWC, w KRSC), or None for a linear
    layer y = x w with x [batch, in_features], w [in_features, out_features]."""

    def __init__(self, conv=None, batch=0, in_features=0, out_features=0, relu=False, seed=0,
                 tensor_id8=1, tensor_id16=2, device="cuda", input_from: "QuantizedLayer | None" = None,
                 emit_codes=False, keep_y=True, keep_z=True, keep_g=True):
        """input_from: the layer whose output feeds this one already quantised (it must have been built with
        emit_codes=True): this layer then owns no input codes of its own and its forward takes no fp32 input.
        emit_codes: the forward also writes the 8-bit codes of the output (and each row's code sum) for the next
        layer; keep_y=False then leaves the fp32 output unwritten.  keep_z=False (forward only, with emit_codes and
        keep_y=False): the fp32 output of the product is not kept either -- the convolution is run twice instead.
        keep_g=False: the backward pass does not write the fp32 gradient arriving at the product (only its 8-bit and
        16-bit copies); for shapes the library quantises as it computes the gradient (it says so otherwise)."""
        self.device = torch.device(device)
        d = B.LayerDesc()
        if conv is not None:
            d.conv = conv
            self.rows, self.cin, self.cout = conv.N * conv.H * conv.W, conv.C, conv.K
            self.x_shape = (conv.N, conv.H, conv.W, conv.C)
            self.w_shape = (conv.K, conv.R, conv.S, conv.C)
            self.z_shape = (conv.N, conv.H, conv.W, conv.K)
        else:
            d.batch, d.in_features, d.out_features = batch, in_features, out_features
            self.rows, self.cin, self.cout = batch, in_features, out_features
            self.x_shape, self.w_shape, self.z_shape = (batch, in_features), (in_features, out_features), (batch, out_features)
        d.relu, d.seed, d.tensor_id8, d.tensor_id16 = int(relu), seed, tensor_id8, tensor_id16
        self.desc = d
        dev = self.device
        e = lambda shape, dt: torch.empty(shape, dtype=dt, device=dev)
        self.w_codes = e(self.w_shape, torch.int8)
        self.qw, self.qg8, self.qg16 = (B.new_qparams(1, dev) for _ in range(3))
        self.rq_in = None
        if input_from is not None:
            assert input_from.rq_out is not None and input_from.z_shape == self.x_shape
            self.x_codes, self.qx = input_from.out_codes, input_from.q_out
            self.rq_in = input_from.rq_out
            self.x_chan_sums = input_from.out_chan_sums
        else:
            self.x_codes, self.qx = e(self.x_shape, torch.int8), B.new_qparams(1, dev)
            self.x_chan_sums = e((self.cin,), torch.int64) if conv is not None and self.rows < (1 << 22) else None
        self.rq_out = None
        if emit_codes:
            self.out_codes, self.q_out = e(self.z_shape, torch.int8), B.new_qparams(1, dev)
            self.out_row_sums = e((self.rows,), torch.int32)
            self.out_chan_sums = e((self.cout,), torch.int64) if conv is not None and self.rows < (1 << 22) else None
            self.rq_out = B.requant(self.out_codes, self.q_out, self.out_row_sums, self.out_chan_sums)
        assert keep_z or (emit_codes and not keep_y)
        self.z = e(self.z_shape, torch.float32) if keep_z else None
        self.g = e(self.z_shape, torch.float32) if (keep_z and keep_g) else None
        self.save_mean, self.save_min, self.save_max = (e((self.cout,), torch.float32) for _ in range(3))
        bshape = self.z_shape if keep_z else (0,)          # (no backward pass without z)
        self.g8, self.ghi, self.glo = e(bshape, torch.int8), e(bshape, torch.int8), e(bshape, torch.uint8)
        assert keep_y or emit_codes
        self.y = e(self.z_shape, torch.float32) if keep_y else None
        self.dx, self.dw = e(self.x_shape, torch.float32), e(self.w_shape, torch.float32)
        self.dgamma, self.dbeta = e((self.cout,), torch.float32), e((self.cout,), torch.float32)
        self.ws = torch.empty(max(B.qbp_layer_workspace_bytes(d), 256), dtype=torch.uint8, device=dev)
        c = B.LayerCtx()
        for name, t in (("x_codes", self.x_codes), ("qx", self.qx), ("w_codes", self.w_codes), ("qw", self.qw),
                        ("z", self.z), ("save_mean", self.save_mean), ("save_min", self.save_min),
                        ("save_max", self.save_max), ("g", self.g), ("g8", self.g8), ("qg8", self.qg8),
                        ("g_hi", self.ghi), ("g_lo", self.glo), ("qg16", self.qg16), ("x_chan_sums", self.x_chan_sums)):
            setattr(c, name, t.data_ptr() if t is not None and t.numel() else None)
        self.ctx = c
        self.gamma = self.beta = None

    def forward(self, x, w, gamma=None, beta=None):
        """x: the fp32 input, or None for a layer built with input_from (its input codes are already there)."""
        self.gamma, self.beta = gamma, beta
        assert (x is None) == (self.rq_in is not None)
        if self.rq_in is None and self.rq_out is None:
            return B.qbp_layer_fwd(self.desc, x, w, gamma, beta, self.y, self.ctx, self.ws)
        return B.qbp_layer_fwd_chained(self.desc, x, self.rq_in, w, gamma, beta, self.y, self.rq_out, self.ctx, self.ws)

    def backward(self, dy):
        return B.qbp_layer_bwd(self.desc, self.ctx, dy, self.gamma, self.beta, self.dx, self.dw, self.dgamma,
                               self.dbeta, self.ws)

    def status(self) -> int:
        return B.status_word(self.ws)


class QuantizedStack:
    """A chain of quantised convolution layers, each followed by Range BN + ReLU, trained as the method prescribes
    (Sections 4 and 6): every inner activation is handed on as the 8-bit codes its Range BN wrote (no range scan and
    no quantisation pass between layers), gradients flow back through qbp_layer_bwd, and the fp32 master weights,
    gamma and beta are updated once per minibatch by qbp_sgd_update.  Buffer bookkeeping and call order only."""

    def __init__(self, convs, weights, seed=0, chained=True, keep_y=False, lr=0.1, momentum=0.9, weight_decay=1e-4,
                 device="cuda"):
        """convs: binding.ConvDesc per layer (layer i's output shape = layer i+1's input shape); weights: the fp32
        master weights (KRSC device tensors, updated in place).  chained=False runs every layer from the fp32
        activation of the one before (range scan + quantiser per layer) -- the unfused composition, for comparison."""
        self.chained, self.lr, self.momentum, self.weight_decay = chained, lr, momentum, weight_decay
        self.w = list(weights)
        self.layers = []
        n = len(convs)
        for i, conv in enumerate(convs):
            last = i == n - 1
            prev = self.layers[-1] if (self.layers and chained) else None
            self.layers.append(QuantizedLayer(conv=conv, relu=True, seed=seed, tensor_id8=i + 1, tensor_id16=i + 1, device=device,
                                              input_from=prev, emit_codes=chained and not last,
                                              keep_y=(not chained) or last or keep_y))
        dev = torch.device(device)
        self.gamma = [torch.ones(L.cout, dtype=torch.float32, device=dev) for L in self.layers]
        self.beta = [torch.zeros(L.cout, dtype=torch.float32, device=dev) for L in self.layers]
        mk = lambda ts: [torch.zeros_like(t) for t in ts] if momentum else [None] * len(ts)
        self.vw, self.vg, self.vb = mk(self.w), mk(self.gamma), mk(self.beta)

    def forward(self, x):
        a = x
        for L, w, g, b in zip(self.layers, self.w, self.gamma, self.beta):
            y = L.forward(a if L.rq_in is None else None, w, g, b)
            a = y
        return self.layers[-1].y

    def backward(self, dy):
        d = dy
        for L in reversed(self.layers):
            d, _, _, _ = L.backward(d)         # dx of a layer is the gradient at the previous layer's output
        return d

    def update(self):
        for L, w, g, b, vw, vg, vb in zip(self.layers, self.w, self.gamma, self.beta, self.vw, self.vg, self.vb):
            B.qbp_sgd_update(w, L.dw, vw, self.lr, self.momentum, self.weight_decay)
            B.qbp_sgd_update(g, L.dgamma, vg, self.lr, self.momentum, 0.0)
            B.qbp_sgd_update(b, L.dbeta, vb, self.lr, self.momentum, 0.0)

    def train_step(self, x, dy):
        self.forward(x)
        dx = self.backward(dy)
        self.update()
        return dx

    def status(self) -> int:
        return min(L.status() for L in self.layers)


class TernarizedLayer:
    """The low-bit form of the quantised layer (Appendix C, Ternarized Back-Propagation): 1-bit weights and activations,
    a ternary gradient for the layer-gradient product, and Algorithm 1 (the mean over `samples` ternarisations) for the
    weight gradient; Range BN after the product as in the 8-bit layer.  Call order and buffers only: binarise x and w
    -> product (the +-1 dot product of XNOR + popcount, on the int8 tensor cores) -> Range BN; backwards Range BN ->
    ternarise the gradient -> layer-gradient product; ternarise `samples` times -> weight-gradient product."""

    def __init__(self, conv=None, relu=False, seed=0, tensor_id=1, samples=1):
        self.conv, self.relu, self.seed, self.tensor_id, self.samples = conv, relu, seed, tensor_id, samples
        self.saved = None

    def forward(self, x, w, gamma=None, beta=None):
        a, qa = B.qbp_binarize_s8(x)
        wb, qw = B.qbp_binarize_s8(w)
        if self.conv is not None:
            _, z, _ = B.qbp_conv_s8_implicit(B.QBP_CONV_FPROP, self.conv, a, qa, wb, qw)
        else:
            _, z, _ = B.qbp_gemm_s8(a, qa, wb, qw)                     # x [batch x in] . w [in x out]
        y, mean, vmin, vmax, _ = B.qbp_rangebn_fwd(z, gamma, beta, relu=self.relu)
        self.saved = dict(a=a, qa=qa, wb=wb, qw=qw, z=z, mean=mean, vmin=vmin, vmax=vmax, gamma=gamma, beta=beta)
        return y

    def backward(self, dy):
        s = self.saved
        g, dgamma, dbeta = B.qbp_rangebn_bwd(dy, s["z"], s["mean"], s["vmin"], s["vmax"], s["gamma"], s["beta"], relu=self.relu)
        # sample 0 of the gradient's stream serves the layer gradient; the weight gradient draws its own samples
        t, qt = B.qbp_stc_ternarize_s8(g, samples=1, seed=self.seed, tensor_id=self.tensor_id)
        if self.conv is not None:
            _, dx, _ = B.qbp_conv_s8_implicit(B.QBP_CONV_DGRAD, self.conv, t, qt, s["wb"], s["qw"])
        else:
            _, dx, _ = B.qbp_gemm_s8(t, qt, s["wb"], s["qw"], transB=True)
        _, dw, _, _, _ = B.qbp_tbp_weight_gradient(s["a"], s["qa"], g, self.samples, seed=self.seed, tensor_id=self.tensor_id + 1,
                                                   d=self.conv)
        self.g, self.t, self.qt = g, t, qt
        return dx, dw, dgamma, dbeta
