"""One training step of a CDL quantized layer as a fixed sequence of C-ABI calls (Algorithm 1, the
per-layer part of its forward and backward passes).  This module only owns device buffers and issues the
calls in order on one stream; every number is produced by the kernels behind the ABI.

Step (names follow the paper: w weights, x activations, q / s step sizes, alpha / beta CPMF parameters):
   1  quantize w        -> soft value Q_d(w), index W_idx, level histogram          cdl_quantize_soft
   2  entropy of w      -> H(w) in bits, level probabilities                        cdl_index_entropy
   3  quantize x        -> Q_d(x), index X_idx, histogram (window of 5)             cdl_quantize_soft
   4  entropy of x                                                                   cdl_index_entropy
   5  forward product   Y = (s q) A_idx W_idx   (A_idx: the im2col index matrix)    cdl_qlinear_fwd
   6  quantize dL/dY    -> G_idx (hard index, 255 levels, caller-chosen step)       cdl_quantize_hard
   7  backward products dA = (q_g q) G_idx W_idx^T, dW = (q_g s) A_idx^T G_idx      cdl_qlinear_bwd (two calls)
   8  quantizer backward on x: dL/dx, dL/ds, dL/dbeta (+ gamma * rate term)         cdl_quantize_backward
   9  quantizer backward on w with grad_out = dW: dL/dw, dL/dq, dL/dalpha (+ lambda * rate term)
The im2col gather / scatter between the activation tensor and the GEMM operand is outside the library:
A_idx and the gradient arriving at the quantized activations are inputs of the step.

Data-parallel ranks pass run(exchange=StepExchange): the activation histogram is then summed over the ranks before
step 4, the weight-gradient product of step 7 delivers its int32 accumulators, which are summed over the ranks and
converted to float once (cdl_rescale_acc), and the two scalar gradients of the activation quantizer are summed at
the end; everything that depends on the weights alone is identical on every rank and is not exchanged.

With conv=ConvShape(...) the layer is a convolution (any stride and padding cdl_qconv_* takes) computed straight from the NHWC index tensor
(cdl_qconv_fwd / cdl_qconv_bwd): steps 5 and 7 read X_idx itself, dA becomes dL/dQ(x) in the layout of x, and step 8
takes it as its incoming gradient, so the only inputs of a step are w, x and dL/dY.
"""
from __future__ import annotations

from . import api as cdl

CALLS = ("quantize_soft_w", "entropy_w", "quantize_soft_x", "entropy_x", "qlinear_fwd", "quantize_hard_g",
         "qlinear_bwd_dx", "qlinear_bwd_dw", "quantize_backward_x", "quantize_backward_w")


class CdlLayerStep:
    def __init__(self, torch, M, K, N, n_x, wq, xq, q_g, device="cuda", lda=None, need_dx=True, conv=None):
        """wq / xq: objects with q, lo, hi, alpha, rate_weight, window (weights / activations); n_x: number of
        activation elements quantized per step (the layer's input tensor, before im2col); conv: a ConvShape for
        the convolution form (then M = N*P*Q output pixels, K = R*S*C, n_x = N*H*W*C input elements)."""
        self.torch = torch
        self.conv = conv
        if conv is not None:
            assert M == conv.N * conv.P * conv.Q and K == conv.R * conv.S * conv.C
            assert n_x == conv.N * conv.H * conv.W * conv.C
        self.M, self.K, self.N, self.n_x, self.n_w = M, K, N, n_x, K * N
        self.need_dx = need_dx      # False for the first layer of a network: its input needs no gradient
        self.lda = lda if lda is not None else (K + 15) // 16 * 16     # row pitch of A_idx (multiple of 16 bytes)
        self.wq, self.xq, self.q_g = wq, xq, float(q_g)
        t, dev = torch, device
        f32, i8, u8 = t.float32, t.int8, t.uint8

        def idt(lo):
            return i8 if lo < 0 else u8
        # inputs of a step
        self.w = t.empty(self.n_w, dtype=f32, device=dev)
        self.x = t.empty(n_x, dtype=f32, device=dev)
        self.A_idx = t.zeros((M, self.lda), dtype=idt(xq.lo), device=dev) if conv is None else None
        self.dY = t.empty((M, N), dtype=f32, device=dev)
        # dL/dQ(x): an input after the scatter back from dA, or the convolution's own data gradient
        self.gx_in = t.empty(n_x, dtype=f32, device=dev)
        # outputs
        self.w_soft = t.empty(self.n_w, dtype=f32, device=dev)
        self.W_idx = t.empty((K, N), dtype=idt(wq.lo), device=dev)
        self.x_soft = t.empty(n_x, dtype=f32, device=dev)
        self.X_idx = t.empty(n_x, dtype=idt(xq.lo), device=dev)
        self.hist_w = t.zeros(wq.hi - wq.lo + 1, dtype=t.int64, device=dev)
        self.hist_x = t.zeros(xq.hi - xq.lo + 1, dtype=t.int64, device=dev)
        self.prob_w = t.empty(wq.hi - wq.lo + 1, dtype=f32, device=dev)
        self.prob_x = t.empty(xq.hi - xq.lo + 1, dtype=f32, device=dev)
        self.Y = t.empty((M, N), dtype=f32, device=dev)
        self.G_idx = t.empty((M, N), dtype=i8, device=dev)
        self.dA = (t.empty((M, K), dtype=f32, device=dev) if need_dx else None) if conv is None else self.gx_in
        self.dW = t.empty((K, N), dtype=f32, device=dev)
        self.dx = t.empty(n_x, dtype=f32, device=dev)
        self.dw = t.empty(self.n_w, dtype=f32, device=dev)
        # scalars: H(w), H(x) | dq, dalpha, ds, dbeta
        self.scalars = t.zeros(6, dtype=t.float64, device=dev)
        if conv is None:
            self.ws_bytes = max(cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_FWD, M, N, K),
                                cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_BWD, M, N, K))
        else:
            self.ws_bytes = cdl.cdl_qconv_workspace_bytes(conv, N)
            assert self.ws_bytes > 0, "convolution shape not supported by cdl_qconv_*"
        self.ws = t.empty(self.ws_bytes, dtype=u8, device=dev)
        self.Pw = cdl.QuantParams(wq.q, wq.lo, wq.hi, wq.alpha, wq.rate_weight, None, wq.window)
        self.Px = cdl.QuantParams(xq.q, xq.lo, xq.hi, xq.alpha, xq.rate_weight, None, xq.window)
        self.Pw_b = cdl.QuantParams(wq.q, wq.lo, wq.hi, wq.alpha, wq.rate_weight, self.prob_w, wq.window)
        self.Px_b = cdl.QuantParams(xq.q, xq.lo, xq.hi, xq.alpha, xq.rate_weight, self.prob_x, xq.window)
        self.Pg = cdl.QuantParams(self.q_g, -127, 127)
        self.da = cdl.IndexDesc(xq.q, xq.lo, xq.hi)
        self.dw_desc = cdl.IndexDesc(wq.q, wq.lo, wq.hi)
        self.dg = cdl.IndexDesc(self.q_g, -127, 127)

    def kernels_per_step(self):
        """Kernels of this library one step launches: one per call, plus the small kernel that turns the split
        weight-gradient reduction into floats when the reduction over M is split across SMs."""
        split_dw = self.ws_bytes > 256
        return len(CALLS) - (0 if self.need_dx else 1) + (1 if split_dw else 0)

    def capture(self, concurrent=True):
        """Record one step into a CUDA graph and return it (``graph.replay()`` enqueues the step on the current
        stream).  All buffers of a step are owned by this object and never reallocated, so the recorded pointers
        stay valid.  One step runs eagerly first: the library's one-time set-up per device must not fall into the
        capture.  With concurrent=True the calls are recorded on three streams along the data dependencies of the
        step (see run_forked), so that the short kernels run beside the long ones."""
        t = self.torch
        graph = t.cuda.CUDAGraph()
        side = t.cuda.Stream()
        side.wait_stream(t.cuda.current_stream())
        with t.cuda.stream(side):
            self.run()
            side.synchronize()
            with t.cuda.graph(graph, stream=side):
                if concurrent:
                    self.run_forked()
                else:
                    self.run()
        t.cuda.current_stream().wait_stream(side)
        return graph

    def run_forked(self):
        """The same ten calls as run(), issued on the current stream and two helper streams along the step's data
        dependencies.  Stored-matrix form:
            current:  dW -> forward -> dA                       (the three products, back to back)
            second:   quantize x -> entropy of x -> quantizer backward on x
            third:    quantize dL/dY -> quantize w -> entropy of w -> quantizer backward on w
        dW needs G_idx but not W_idx, so it goes first and the weight passes leave the chain of the products (the
        forward product needs W_idx, dA needs G_idx and W_idx, the backward pass on w needs dW and the level
        probabilities of w and runs beside the other two products).  Convolution form, where the forward product
        and dW read X_idx and the activation quantizer's backward pass reads dA:
            current:  quantize w -> forward -> dA -> dW -> quantizer backward on w
            second:   quantize x -> entropy of x -> (after dA) quantizer backward on x
            third:    quantize dL/dY ;  entropy of w
        Both orders are the fastest of the alternatives measured on a ResNet-18 layer3 convolution (a product occupies
        every SM while it runs, so what overlaps with what is decided by the order); all helper work is joined back
        into the current stream at the end."""
        t = self.torch
        if not hasattr(self, "_helpers"):
            self._helpers = (t.cuda.Stream(), t.cuda.Stream())
        s0 = t.cuda.current_stream()
        s1, s2 = self._helpers
        sc = self.scalars
        M, K, N = self.M, self.K, self.N
        nlw, nlx = self.Pw.nlev, self.Px.nlev

        def after(stream):
            e = t.cuda.Event()
            e.record(stream)
            return e
        fork = after(s0)
        s1.wait_event(fork)
        s2.wait_event(fork)
        # second stream: everything on the activation tensor
        cdl.cdl_quantize_soft(self.x, self.n_x, self.Px, self.x_soft, self.X_idx, self.hist_x, s1)
        x_ready = after(s1)
        cdl.cdl_index_entropy(self.hist_x, nlx, sc[1:2], self.prob_x, None, s1)
        if self.conv is None:
            cdl.cdl_quantize_backward(self.x, self.gx_in, self.n_x, self.Px_b, self.dx, sc[4:5], sc[5:6], s1)
            # third stream: gradient indices first (dW waits for them), then the weights
            cdl.cdl_quantize_hard(self.dY, M * N, self.Pg, self.G_idx, None, s2)
            g_ready = after(s2)
            cdl.cdl_quantize_soft(self.w, self.n_w, self.Pw, self.w_soft, self.W_idx, self.hist_w, s2)
            w_ready = after(s2)
            cdl.cdl_index_entropy(self.hist_w, nlw, sc[0:1], self.prob_w, None, s2)
            # current stream: the three products
            s0.wait_event(g_ready)
            self._bwd_dw(s0)
            dw_ready = after(s0)
            s0.wait_event(w_ready)
            self._fwd(s0)
            self._bwd_dx(s0)
            s2.wait_event(dw_ready)
            cdl.cdl_quantize_backward(self.w, self.dW, self.n_w, self.Pw_b, self.dw, sc[2:3], sc[3:4], s2)
        else:
            # third stream: gradient indices
            cdl.cdl_quantize_hard(self.dY, M * N, self.Pg, self.G_idx, None, s2)
            g_ready = after(s2)
            # current stream: weights, then the three products
            cdl.cdl_quantize_soft(self.w, self.n_w, self.Pw, self.w_soft, self.W_idx, self.hist_w, s0)
            w_ready = after(s0)
            s2.wait_event(w_ready)
            cdl.cdl_index_entropy(self.hist_w, nlw, sc[0:1], self.prob_w, None, s2)
            s0.wait_event(x_ready)
            self._fwd(s0)
            s0.wait_event(g_ready)
            self._bwd_dx(s0)
            s1.wait_event(after(s0))
            cdl.cdl_quantize_backward(self.x, self.gx_in, self.n_x, self.Px_b, self.dx, sc[4:5], sc[5:6], s1)
            self._bwd_dw(s0)
            s0.wait_event(after(s2))
            cdl.cdl_quantize_backward(self.w, self.dW, self.n_w, self.Pw_b, self.dw, sc[2:3], sc[3:4], s0)
        s0.wait_event(after(s1))
        s0.wait_event(after(s2))

    def input_tensors(self):
        if self.conv is not None:
            return {"w": self.w, "x": self.x, "dY": self.dY}
        return {"w": self.w, "x": self.x, "A_idx": self.A_idx, "dY": self.dY, "gx_in": self.gx_in}

    # the three products, in either form
    def _fwd(self, stream):
        M, K, N = self.M, self.K, self.N
        if self.conv is None:
            cdl.cdl_qlinear_fwd(self.A_idx, self.lda, self.da, self.W_idx, N, self.dw_desc, M, N, K, None, self.Y,
                                None, self.ws, self.ws_bytes, stream)
        else:
            cdl.cdl_qconv_fwd(self.X_idx, self.da, self.W_idx, N, self.dw_desc, self.conv, N, None, self.Y, None,
                              self.ws, self.ws_bytes, stream)

    def _bwd_dx(self, stream):
        M, K, N = self.M, self.K, self.N
        if not self.need_dx:
            return
        if self.conv is None:
            cdl.cdl_qlinear_bwd(self.G_idx, N, self.dg, None, K, None, self.W_idx, N, self.dw_desc,
                                M, N, K, None, self.dA, None, None, self.ws, self.ws_bytes, stream)
        else:
            cdl.cdl_qconv_bwd(self.G_idx, self.dg, None, None, self.W_idx, N, self.dw_desc, self.conv, N,
                              None, self.dA, None, None, self.ws, self.ws_bytes, stream)

    def _bwd_dw(self, stream, acc=None):
        """dW as floats, or (acc given) as int32 accumulators for a later sum over ranks."""
        M, K, N = self.M, self.K, self.N
        dWf = self.dW if acc is None else None
        if self.conv is None:
            cdl.cdl_qlinear_bwd(self.G_idx, N, self.dg, self.A_idx, self.lda, self.da, None, N, None,
                                M, N, K, None, None, acc, dWf, self.ws, self.ws_bytes, stream)
        else:
            cdl.cdl_qconv_bwd(self.G_idx, self.dg, self.X_idx, self.da, None, N, None, self.conv, N,
                              None, None, acc, dWf, self.ws, self.ws_bytes, stream)

    def _bwd_dw_exchanged(self, stream, exchange, rows_global):
        """Weight gradient of the global batch: local integer accumulators, summed over the ranks as integers,
        one conversion to float afterwards - the bits of a single product over all rows."""
        from . import sharding
        t = self.torch
        if not hasattr(self, "dWacc"):
            self.dWacc = t.empty((self.K, self.N), dtype=t.int32, device=self.dW.device)
        self._bwd_dw(stream, acc=self.dWacc)
        amax = max(abs(self.xq.lo), abs(self.xq.hi))
        bits = sharding.acc_bits_for(rows_global, amax, 127)
        acc = self.dWacc if bits == 32 else self.dWacc.to(t.int64)
        exchange.accumulators(acc)
        cdl.cdl_rescale_acc(acc, bits, self.K * self.N, self.q_g, self.xq.q, self.dW, stream)

    def run(self, stream=None, mark=None, exchange=None, rows_global=None):
        """Enqueue one step.  mark(name), if given, is called before each ABI call and once at the end
        (used to drop CUDA events between the calls).  exchange: a sharding.StepExchange when this rank holds a block
        of the batch rows (rows_global = rows of all ranks together); the collectives run on the current stream,
        which must then be the stream the calls are enqueued on."""
        s = self.scalars
        M, K, N = self.M, self.K, self.N
        nlw, nlx = self.Pw.nlev, self.Px.nlev
        m = mark if mark is not None else (lambda name: None)
        m(CALLS[0]); cdl.cdl_quantize_soft(self.w, self.n_w, self.Pw, self.w_soft, self.W_idx, self.hist_w, stream)
        m(CALLS[1]); cdl.cdl_index_entropy(self.hist_w, nlw, s[0:1], self.prob_w, None, stream)
        m(CALLS[2]); cdl.cdl_quantize_soft(self.x, self.n_x, self.Px, self.x_soft, self.X_idx, self.hist_x, stream)
        if exchange is not None:
            exchange.histogram(self.hist_x)          # level counts of the whole batch, before H(x) and prob_x
        m(CALLS[3]); cdl.cdl_index_entropy(self.hist_x, nlx, s[1:2], self.prob_x, None, stream)
        m(CALLS[4]); self._fwd(stream)
        m(CALLS[5]); cdl.cdl_quantize_hard(self.dY, M * N, self.Pg, self.G_idx, None, stream)
        # the two backward products are issued as two calls so that each can be timed on its own
        m(CALLS[6]); self._bwd_dx(stream)
        m(CALLS[7])
        if exchange is None:
            self._bwd_dw(stream)
        else:
            self._bwd_dw_exchanged(stream, exchange, rows_global if rows_global is not None else M * exchange.world)
        m(CALLS[8]); cdl.cdl_quantize_backward(self.x, self.gx_in, self.n_x, self.Px_b, self.dx, s[4:5], s[5:6], stream)
        m(CALLS[9]); cdl.cdl_quantize_backward(self.w, self.dW, self.n_w, self.Pw_b, self.dw, s[2:3], s[3:4], stream)
        if exchange is not None:
            exchange.batch_scalars(s[4:6])           # dL/ds, dL/dbeta: sums over the batch; the rest is replicated
        m("end")
