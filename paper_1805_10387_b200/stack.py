"""One mixed-precision training step of a stack of linear layers, as a sequence of calls
into the C-ABI library.  This module only owns device buffers and orders the calls; it does
no arithmetic.

Order of one step (paper Section 3.1-3.2): forward products bottom-up; the FP32 gradient
entering each top layer is multiplied by the current loss scale S on the device; backward
products top-down (the weight-gradient kernels inspect what they store and raise the
device flag); one fused master update over all layers, which writes nothing when the flag
is set; the loss-scale state machine picks S for the next step.  Nothing returns to the
host inside a step.
"""
from __future__ import annotations

import contextlib

import torch

from . import dp, mp


def _align(n: int, a: int = 8) -> int:
    return (n + a - 1) // a * a


class LinearStack:
    def __init__(self, shapes, chained, optimizer="adam", lr=1e-3, beta1=0.9, beta2=0.999,
                 eps=1e-8, momentum=0.9, weight_decay=0.0, init_scale=65536.0,
                 growth_interval=1000, min_scale=1.0, max_scale=2.0 ** 24, dynamic=True,
                 device="cuda", acts=None, clip=20.0, bias=False, overflow_tolerance=1, lstm=None,
                 comm=None, shard_update=False, overlap_wgrad=None):
        """acts[l]: mp.MP_ACT_* after layer l's product (a layer whose output feeds no chained
        layer must have MP_ACT_NONE); bias: every layer gets a bias vector; lstm[l]: layer l's
        product is the gate pre-activation of an LSTM cell (N = 4 H, gate order i, f, g, o): the
        cell kernels turn it and the cell state c_prev[l] into c_new[l] and h[l], the gradient
        entering the layer is that of h ([M, H]), and the cell's backward kernel produces the
        gate gradient that the layer's two backward products consume.
        comm: data-parallel exchange (an object with the methods of dp.Comm; None = one rank).
        shard_update: with a comm of G ranks, each rank keeps and updates only its 1/G slice of
        the FP32 master and moments (reduce-scatter of the gradients before, all-gather of the
        FP16 weights after) instead of every rank repeating the whole update."""
        self.shapes = [tuple(s) for s in shapes]
        self.chained = list(chained)
        self.L = len(shapes)
        self.acts = list(acts) if acts is not None else [mp.MP_ACT_NONE] * self.L
        self.clip, self.has_bias = float(clip), bool(bias)
        self.lstm = list(lstm) if lstm is not None else [False] * self.L
        for l in range(self.L):
            if self.lstm[l]:
                assert self.shapes[l][2] % 32 == 0 and self.acts[l] == mp.MP_ACT_NONE and not self.has_bias
                assert not (l + 1 < self.L and self.chained[l + 1]), "an LSTM layer's gates feed no other layer"
        for l in range(self.L):
            feeds = l + 1 < self.L and self.chained[l + 1]
            assert feeds or self.acts[l] == mp.MP_ACT_NONE, "a top layer has no activation"
        self.device = torch.device(device)
        self.opt = mp.OptimConfig(mp.MP_OPT_ADAM if optimizer == "adam" else mp.MP_OPT_MOMENTUM,
                                  lr, beta1, beta2, eps, momentum, weight_decay)
        self.state = mp.State(init_scale, growth_interval, min_scale, max_scale, dynamic,
                              overflow_tolerance)

        # parameters, moments and weight gradients live in flat buffers; every tensor starts on
        # a 16-byte boundary and rows are padded to a multiple of 8 elements
        self.ldw = [_align(n) for _, _, n in self.shapes]
        sizes = [k * ld for (_, k, _), ld in zip(self.shapes, self.ldw)]
        offs, total = [], 0
        for s in sizes:
            offs.append(total)
            total += _align(s)
        boffs = []                                   # biases follow the weights in the same buffers
        for _, _, n in self.shapes:
            boffs.append(total)
            total += _align(n) if self.has_bias else 0
        self.comm = comm
        self.world = comm.world if comm is not None else 1
        self.rank = comm.rank if comm is not None else 0
        self.shard_update = bool(shard_update) and self.world > 1
        if self.shard_update:
            # equal slices that start on 16-byte boundaries: pad the flat range to 8 * world elements
            total = dp.padded_total(total, self.world)
        self.offsets, self.boffsets, self.sizes, self.total = offs, boffs, sizes, total
        f16 = dict(dtype=torch.float16, device=self.device)
        f32 = dict(dtype=torch.float32, device=self.device)
        self.w16_flat = torch.zeros(total, **f16)
        self.dw_flat = torch.zeros(total, **f16)
        view = lambda flat, l: flat[offs[l]:offs[l] + sizes[l]].view(self.shapes[l][1], self.ldw[l])
        bview = lambda flat, l: flat[boffs[l]:boffs[l] + self.shapes[l][2]] if self.has_bias else None
        self.w16 = [view(self.w16_flat, l) for l in range(self.L)]
        self.dw = [view(self.dw_flat, l) for l in range(self.L)]
        self.b16 = [bview(self.w16_flat, l) for l in range(self.L)]
        self.db = [bview(self.dw_flat, l) for l in range(self.L)]
        if not self.shard_update:
            self.shard = (0, total)
            self.w32_flat = torch.zeros(total, **f32)
            self.m_flat = torch.zeros(total, **f32)
            self.v_flat = torch.zeros(total, **f32) if optimizer == "adam" else None
            self.w32 = [view(self.w32_flat, l) for l in range(self.L)]
            self.m = [view(self.m_flat, l) for l in range(self.L)]
            self.v = [view(self.v_flat, l) for l in range(self.L)] if self.v_flat is not None else None
            self.b32 = [bview(self.w32_flat, l) for l in range(self.L)]
            # one plan over the whole flat range: padding columns hold zeros and stay zero
            self.plan = mp.UpdatePlan([self.dw_flat], [self.w32_flat], [self.m_flat],
                                      [self.v_flat] if self.v_flat is not None else None,
                                      [self.w16_flat])
        else:
            # this rank's slice [lo, hi) of the flat parameter range: the only part of the FP32
            # master and of the moments that exists here
            lo, hi = self.shard = dp.shard_params(total, self.rank, self.world)
            n = hi - lo
            self.w32_flat = torch.zeros(n, **f32)
            self.m_flat = torch.zeros(n, **f32)
            self.v_flat = torch.zeros(n, **f32) if optimizer == "adam" else None
            self.w32 = self.m = self.v = self.b32 = None      # per-layer FP32 views do not exist
            self.dw_shard = torch.zeros(n, **f16)             # reduced gradients of the slice
            self.flag_word = torch.zeros(1, dtype=torch.int32, device=self.device)
            self.plan = mp.UpdatePlan([self.dw_shard], [self.w32_flat], [self.m_flat],
                                      [self.v_flat] if self.v_flat is not None else None,
                                      [self.w16_flat[lo:lo + n]])

        # activations and their gradients
        self.x = [None] * self.L
        self.y = [torch.empty(m, _align(n), **f16) for m, _, n in self.shapes]
        self.dy = [None] * self.L
        self.dx = [torch.empty(m, _align(k), **f16) for m, k, _ in self.shapes]
        # Scaled upstream gradients of the top layers whose rows need no padding share one flat
        # buffer (ascending layer order): when their FP32 gradients arrive as consecutive slices
        # of one buffer too, a single scaling call covers all of them.
        # (For an LSTM layer the scaled gradient is that of h, [M, H]; its gate gradient has a
        # buffer of its own.)
        self.up_width = [n // 4 if self.lstm[l] else n for l, (_, _, n) in enumerate(self.shapes)]
        self.flat_tops = [l for l in range(self.L) if not (l + 1 < self.L and self.chained[l + 1])
                          and self.up_width[l] % 8 == 0]
        self.dy_top_flat = torch.zeros(sum(self.shapes[l][0] * self.up_width[l] for l in self.flat_tops), **f16)
        flat_off = {}
        o = 0
        for l in self.flat_tops:
            flat_off[l] = o
            o += self.shapes[l][0] * self.up_width[l]
        self.c_prev, self.c_new, self.h, self.dh, self.dc_prev = ([None] * self.L for _ in range(5))
        for l in range(self.L):
            if self.chained[l]:
                self.x[l] = self.y[l - 1]
            feeds = l + 1 < self.L and self.chained[l + 1]
            if feeds:
                self.dy[l] = self.dx[l + 1]
            elif self.lstm[l]:
                m, _, n = self.shapes[l]
                hh = n // 4
                self.dy[l] = torch.zeros(m, n, **f16)
                self.dh[l] = self.dy_top_flat[flat_off[l]:flat_off[l] + m * hh].view(m, hh)
                self.c_prev[l], self.c_new[l], self.h[l], self.dc_prev[l] = (torch.zeros(m, hh, **f16)
                                                                             for _ in range(4))
            elif l in flat_off:
                m, _, n = self.shapes[l]
                self.dy[l] = self.dy_top_flat[flat_off[l]:flat_off[l] + m * n].view(m, n)
            else:
                self.dy[l] = torch.zeros(self.shapes[l][0], _align(self.shapes[l][2]), **f16)
        # Launch groups.  A layer's level is its depth in its chain (0 for a layer that reads an input of
        # the stack).  Layers of one level do not depend on one another, so those of them that have one
        # shape, one activation and the same kind of neighbours go to the grouped calls, a few layers per
        # launch: a product too small to fill the GPU's waves on its own then shares a persistent work
        # list with its peers.  Forward runs the groups level by level, backward in the reverse order.
        gmax = mp.mp_max_group()
        level = [0] * self.L
        for l in range(self.L):
            level[l] = level[l - 1] + 1 if self.chained[l] else 0
        buckets = {}
        for l in range(self.L):
            below = self.acts[l - 1] if self.chained[l] else mp.MP_ACT_NONE
            key = (level[l], self.shapes[l], self.acts[l], self.lstm[l], self.chained[l], self.feeds_next(l), below)
            buckets.setdefault(key, []).append(l)
        self.groups = []
        for key in sorted(buckets, key=lambda k: (k[0], buckets[k][0])):
            ls = buckets[key]
            for i in range(0, len(ls), gmax):
                self.groups.append(ls[i:i + gmax])
        need = 0
        for g in self.groups:
            m, k, n = self.shapes[g[0]]
            for op in (mp.MP_OP_FWD, mp.MP_OP_DGRAD, mp.MP_OP_WGRAD):
                need = max(need, mp.mp_gemm_workspace_bytes_grouped(len(g), m, k, n, op))
        for m, k, n in self.shapes:
            for op in (mp.MP_OP_FWD, mp.MP_OP_DGRAD, mp.MP_OP_WGRAD):
                need = max(need, mp.mp_gemm_workspace_bytes(m, k, n, op))
            if self.has_bias:
                need = max(need, gmax * mp.mp_bias_grad_workspace_bytes(m, n))
        self.workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=self.device)
        # The weight gradients are off the backward pass's critical path (nothing but the update reads
        # them), and a persistent product kernel leaves SMs idle in its last, partly filled wave of
        # tiles: issued on a second stream, a weight gradient's CTAs take the SMs that the data gradient
        # before it has already left, and vice versa.  The second stream has a workspace of its own.
        # Measured on one B200 (whole step, alternating runs): the Transformer-like stack 3.93 -> 3.86 ms, the
        # DeepSpeech2-like chain 1.99 -> 1.955 ms; a stack of independent full-size layers 2.49 -> 2.52 ms
        # (hence the default).
        self.overlap_wgrad = any(self.chained) if overlap_wgrad is None else bool(overlap_wgrad)
        self.side = torch.cuda.Stream(device=self.device) if self.overlap_wgrad else None
        self.workspace_side = torch.empty(max(need, 16), dtype=torch.uint8, device=self.device) \
            if self.overlap_wgrad else self.workspace

    # ---- data movement (no arithmetic) ----
    def load_weights(self, l: int, w32: torch.Tensor, w16: torch.Tensor, b32=None, b16=None):
        """Copies an FP32 master [K,N] and its FP16 working copy (and a bias pair) into the stack."""
        n = self.shapes[l][2]
        self.w16[l][:, :n].copy_(w16)
        if b16 is not None:
            self.b16[l].copy_(b16)
        if not self.shard_update:
            self.w32[l][:, :n].copy_(w32)
            if b32 is not None:
                self.b32[l].copy_(b32)
            return
        # sharded master: keep the part of this tensor that falls into the rank's slice
        lo, hi = self.shard

        def place(dst_off, src_flat):
            a, b = max(lo, dst_off), min(hi, dst_off + src_flat.numel())
            if a < b:
                self.w32_flat[a - lo:b - lo].copy_(src_flat[a - dst_off:b - dst_off])
        k = self.shapes[l][1]
        padded = torch.zeros(k, self.ldw[l], dtype=torch.float32, device=self.device)
        padded[:, :n].copy_(w32)
        place(self.offsets[l], padded.reshape(-1))
        if b32 is not None:
            place(self.boffsets[l], b32.to(self.device, torch.float32).reshape(-1))

    def X(self, l): return self.x[l][:, :self.shapes[l][1]]
    def Y(self, l): return self.y[l][:, :self.shapes[l][2]]
    def dY(self, l): return self.dy[l][:, :self.shapes[l][2]]
    def dX(self, l): return self.dx[l][:, :self.shapes[l][1]]
    def dW(self, l): return self.dw[l][:, :self.shapes[l][2]]
    def W16(self, l): return self.w16[l][:, :self.shapes[l][2]]
    def W32(self, l): return self.w32[l][:, :self.shapes[l][2]]

    def feeds_next(self, l):
        return l + 1 < self.L and self.chained[l + 1]

    # ---- second stream for the weight gradients ----
    def _fork(self):
        """The second stream waits for everything issued so far on the current one."""
        if self.side is not None:
            self.side.wait_stream(torch.cuda.current_stream())

    def _join(self):
        """The current stream waits for everything issued so far on the second one."""
        if self.side is not None:
            torch.cuda.current_stream().wait_stream(self.side)

    def _wgrad_stream(self):
        return torch.cuda.stream(self.side) if self.side is not None else contextlib.nullcontext()

    # ---- optional per-call device timing (CUDA events on the launching stream) ----
    events = None   # set to a list to collect (name, start_event, end_event)

    only = None       # set to a set of call classes to make step() issue only those calls

    def _call(self, name, fn, *args):
        if self.only is not None and name not in self.only:
            return
        if self.events is None:
            fn(*args)
            return
        ext = self._events_external
        a = torch.cuda.Event(enable_timing=True, external=ext)
        b = torch.cuda.Event(enable_timing=True, external=ext)
        a.record()
        fn(*args)
        b.record()
        self.events.append((name, a, b))

    _events_external = False

    # ---- CUDA graph of the step (removes the per-call host cost of ~40 launches per step) ----
    graph = None

    def capture(self, xs, gs, warmup: int = 2):
        """Records one step on the tensors xs / gs into a CUDA graph; replay() then runs it with
        whatever those tensors hold at that time.  Runs `warmup` real steps first (the library's
        one-time set-up calls must not fall inside the capture), so the training state advances
        by that many steps.  The weight-gradient flag, the loss scale and the step count live on
        the device, so a replayed step skips, halves and doubles exactly like an eager one."""
        side = torch.cuda.Stream(device=self.device)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(warmup):
                self.step(xs, gs)
        torch.cuda.current_stream().wait_stream(side)
        saved, self.events = self.events, None
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.step(xs, gs)
        self.events = saved
        self.graph = g
        return g

    def replay(self):
        self.graph.replay()

    def capture_only(self, xs, gs, classes):
        """Records into a CUDA graph only the step's calls of the given classes ("fwd", "dgrad",
        "wgrad", "scale", "update", "scaler"), in the step's order and on the step's buffers.
        Replaying it back to back and dividing the elapsed device time by the number of
        launches gives the average duration of those kernels without any event node or host
        gap between them.  Call capture() first."""
        assert self.graph is not None, "capture() first"
        saved_events, saved_only = self.events, self.only
        self.events, self.only = None, set(classes)
        g = torch.cuda.CUDAGraph()
        try:
            with torch.cuda.graph(g):
                self.step(xs, gs)
        finally:
            self.events, self.only = saved_events, saved_only
        return g

    def capture_timed(self, xs, gs):
        """Records the step once more with an event-record node before and after every C-ABI
        call and returns (graph, [(call class, start event, end event)]).  After a replay has
        finished, start.elapsed_time(end) is the device time of that call inside the replayed
        step: no host launch gaps, unlike events around call-by-call launches.  Every replay
        overwrites the events, so read them before the next one.  Call capture() first (it
        runs the library's one-time set-up outside any capture)."""
        assert self.graph is not None, "capture() first"
        saved = self.events
        self.events, self._events_external = [], True
        g = torch.cuda.CUDAGraph()
        try:
            with torch.cuda.graph(g):
                self.step(xs, gs)
            ev = self.events
        finally:
            self.events, self._events_external = saved, False
        return g, ev

    def step_from_host(self, xs_host, gs_host):
        """The step as a caller with host data makes it: pinned host inputs are copied to the
        device, the step runs (as a CUDA graph once captured on the staging buffers), and the
        loss-scale state comes back to the host."""
        L = self.L
        if not hasattr(self, "_x_in"):
            self._x_in = [None if self.chained[l] else
                          torch.empty(self.shapes[l][0], _align(self.shapes[l][1]), dtype=torch.float16,
                                      device=self.device) for l in range(L)]
            self._g_in = [None if self.feeds_next(l) else
                          torch.empty(self.shapes[l][0], self.shapes[l][2], dtype=torch.float32,
                                      device=self.device) for l in range(L)]
        for l in range(L):
            if self._x_in[l] is not None:
                self._x_in[l][:, :self.shapes[l][1]].copy_(xs_host[l], non_blocking=True)
            if self._g_in[l] is not None:
                self._g_in[l].copy_(gs_host[l], non_blocking=True)
        if self._host_graph is None and self.use_graph_from_host:
            saved, self.graph = self.graph, None
            self.capture(self._x_in, self._g_in, warmup=1)
            self._host_graph, self.graph = self.graph, saved
        if self._host_graph is not None:
            self._host_graph.replay()
        else:
            self.step(self._x_in, self._g_in)
        return self.state.read()

    _host_graph = None
    use_graph_from_host = False

    def _flat_upstream(self, gs):
        """The FP32 gradients of the flat top layers as one tensor, if they are consecutive
        contiguous slices of one buffer in ascending layer order; else None."""
        ls = self.flat_tops
        if len(ls) < 2 or any(gs[l] is None for l in ls):
            return None
        first = gs[ls[0]]
        store, off = first.untyped_storage(), first.storage_offset()
        for l in ls:
            t = gs[l]
            if (t.dtype != torch.float32 or not t.is_contiguous() or t.storage_offset() != off
                    or t.untyped_storage().data_ptr() != store.data_ptr()
                    or t.numel() != self.shapes[l][0] * self.up_width[l]):
                return None
            off += t.numel()
        return torch.empty(0, dtype=torch.float32, device=first.device).set_(
            store, first.storage_offset(), (off - first.storage_offset(),))

    # ---- the step ----
    def step(self, xs, gs):
        """xs[l]: FP16 [M,K] CUDA tensor (row pitch a multiple of 8) for a layer that is not
        chained; gs[l]: contiguous FP32 [M,N] CUDA tensor, the unscaled gradient entering a layer
        whose output feeds no chained layer."""
        self.products(xs, gs)
        self.finish()

    def products(self, xs, gs):
        """The forward and backward products of the step (arguments as for step())."""
        for l in range(self.L):
            if not self.chained[l]:
                self.x[l] = xs[l]
        Xv = lambda l: self.x[l][:, :self.shapes[l][1]]
        for g in self.groups:
            if len(g) > 1 and len({self.x[l].stride(0) for l in g}) == 1:
                if self.has_bias:
                    self._call("fwd", mp.mp_linear_fwd_act_grouped, [Xv(l) for l in g], [self.W16(l) for l in g],
                               [self.b16[l] for l in g], [self.Y(l) for l in g], self.acts[g[0]], self.clip,
                               self.workspace)
                elif self.acts[g[0]] != mp.MP_ACT_NONE:
                    self._call("fwd", mp.mp_linear_fwd_act_grouped, [Xv(l) for l in g], [self.W16(l) for l in g],
                               None, [self.Y(l) for l in g], self.acts[g[0]], self.clip, self.workspace)
                else:
                    self._call("fwd", mp.mp_linear_fwd_grouped, [Xv(l) for l in g], [self.W16(l) for l in g],
                               [self.Y(l) for l in g], self.workspace)
            else:
                for l in g:
                    if self.acts[l] == mp.MP_ACT_NONE and not self.has_bias:
                        self._call("fwd", mp.mp_linear_fwd, Xv(l), self.W16(l), self.Y(l), self.workspace)
                    else:
                        self._call("fwd", mp.mp_linear_fwd_act, Xv(l), self.W16(l), self.b16[l], self.Y(l),
                                   self.acts[l], self.clip, self.workspace)
            for l in g:
                if self.lstm[l]:      # gates -> new cell state and hidden state
                    self._call("cell", mp.mp_lstm_cell_fwd, self.Y(l), self.c_prev[l], self.c_new[l], self.h[l])
        g_flat = self._flat_upstream(gs)
        if g_flat is not None:        # one scaling call for all flat top layers
            self._call("scale", mp.mp_scale_upstream, g_flat, self.dy_top_flat, self.state)
        for g in reversed(self.groups):
            for l in reversed(g):
                if not self.feeds_next(l) and not (g_flat is not None and l in self.flat_tops):
                    n = self.shapes[l][2]
                    if self.lstm[l]:
                        self._call("scale", mp.mp_scale_upstream, gs[l], self.dh[l], self.state)
                    elif self.dy[l].shape[1] == n:
                        self._call("scale", mp.mp_scale_upstream, gs[l], self.dy[l], self.state)
                    elif self.only is None or "scale" in self.only:
                        # padded rows: scale into a dense buffer, then place (copy only)
                        tmp = torch.empty(self.shapes[l][0], n, dtype=torch.float16, device=self.device)
                        mp.mp_scale_upstream(gs[l], tmp, self.state)
                        self.dy[l][:, :n].copy_(tmp)
            for l in reversed(g):
                if self.lstm[l]:      # gradient of h -> gradient of the gate pre-activations
                    self._call("cell", mp.mp_lstm_cell_bwd, self.Y(l), self.c_prev[l], self.c_new[l], self.dh[l],
                               None, self.dY(l), self.dc_prev[l])
            grouped = (len(g) > 1 and len({self.x[l].stride(0) for l in g}) == 1
                       and len({self.dy[l].stride(0) for l in g}) == 1)
            # the activation of the layer below (the same for every layer of a group) masks the data gradient
            below = self.acts[g[0] - 1] if self.chained[g[0]] else mp.MP_ACT_NONE
            self._fork()                                   # the group's dY is complete
            with self._wgrad_stream():
                if grouped:
                    self._call("wgrad", mp.mp_linear_bwd_wgrad_grouped, [Xv(l) for l in g], [self.dY(l) for l in g],
                               [self.dW(l) for l in g], self.state, self.workspace_side)
                    if self.has_bias:
                        self._call("bgrad", mp.mp_bias_grad_grouped, [self.dY(l) for l in g],
                                   [self.db[l] for l in g], self.state, self.workspace_side)
                for l in reversed(g):
                    if not grouped:
                        self._call("wgrad", mp.mp_linear_bwd_wgrad, Xv(l), self.dY(l), self.dW(l), self.state,
                                   self.workspace_side)
                        if self.has_bias:
                            self._call("bgrad", mp.mp_bias_grad, self.dY(l), self.db[l], self.state,
                                       self.workspace_side)
            if grouped and below == mp.MP_ACT_NONE:
                self._call("dgrad", mp.mp_linear_bwd_dgrad_grouped, [self.dY(l) for l in g],
                           [self.W16(l) for l in g], [self.dX(l) for l in g], self.workspace)
                continue
            for l in reversed(g):
                if below == mp.MP_ACT_NONE:
                    self._call("dgrad", mp.mp_linear_bwd_dgrad, self.dY(l), self.W16(l), self.dX(l),
                               self.workspace)
                else:   # the layer below is activated: mask with its stored output (= this layer's input)
                    self._call("dgrad", mp.mp_linear_bwd_dgrad_act, self.dY(l), self.W16(l), Xv(l), self.dX(l),
                               below, self.clip, self.workspace)
        self._join()                                       # every weight gradient is complete

    def finish(self):
        """Everything after the backward products: the gradient exchange of a data-parallel run,
        the fused update and the loss-scale state machine.  The parts are methods of their own
        so that a test can drive several stacks that stand for ranks in lockstep."""
        if self.only is not None:
            self._call("update", mp.mp_master_update, self.plan, self.state, self.opt, 0)
            self._call("scaler", mp.mp_loss_scale_update, self.state)
            return
        self.exchange_gradients()
        self.inspect_exchanged()
        self.apply_update()
        self.publish_weights()
        self._call("scaler", mp.mp_loss_scale_update, self.state)

    def exchange_gradients(self):
        """Data parallel (Section 4 of the paper): the FP16 weight gradients are summed over the
        ranks; replicated update: all-reduce of the flat buffer; sharded update: reduce-scatter,
        each rank receiving the sum of its slice."""
        if self.comm is None:
            return
        if self.shard_update:
            self.comm.reduce_scatter(self.dw_flat, self.dw_shard)
        else:
            self.comm.all_reduce(self.dw_flat)

    def inspect_exchanged(self):
        """Sharded update only: a rank sees just its slice of the summed gradients, so it
        inspects that slice and the ranks agree on the flag with a one-word max-reduction.  (The
        replicated update inspects the whole reduced buffer inside the update call instead; the
        flags the weight-gradient kernels raised on local gradients stay set either way: an inf
        in a local gradient is an inf in the sum.)"""
        if not self.shard_update:
            return
        self._call("check", mp.mp_check_finite, self.dw_shard, self.state)
        mp.mp_state_export_flag(self.state, self.flag_word)
        self.comm.all_reduce_max(self.flag_word)
        mp.mp_state_import_flag(self.state, self.flag_word)

    def apply_update(self):
        # replicated data-parallel update: the call inspects the reduced gradients itself
        self._call("update", mp.mp_master_update, self.plan, self.state, self.opt,
                   1 if (self.comm is not None and not self.shard_update) else 0)

    def publish_weights(self):
        """Sharded update only: every rank rewrote the FP16 copy of its slice; gather the slices."""
        if self.shard_update:
            lo, hi = self.shard
            self.comm.all_gather(self.w16_flat, self.w16_flat[lo:hi])

    def close(self):
        self.plan.close()
        self.state.close()


class HostPipeline:
    """Host-fed steps with the copies of the next batch under the step of the current one.

    Two sets of device staging buffers alternate.  submit() copies one batch from pinned host
    memory into the idle set on a copy stream; run() waits for the oldest submitted batch, runs
    the step on it (a CUDA graph per staging set, recorded the first time the set is used) and
    returns the loss-scale state read back from the device.  With one batch submitted ahead,
        submit(b0); for i: submit(b[i+1]); state = run()
    the host-to-device copy of batch i+1 overlaps the kernels of batch i; every batch is still
    copied and every state still read, only not one after the other.  No arithmetic here."""

    def __init__(self, stack: LinearStack, use_graph: bool = True):
        s = self.stack = stack
        self.use_graph = use_graph
        self.copy_stream = torch.cuda.Stream(device=s.device)
        mk_x = lambda l: None if s.chained[l] else torch.zeros(
            s.shapes[l][0], _align(s.shapes[l][1]), dtype=torch.float16, device=s.device)

        def mk_gs():      # one flat FP32 buffer, sliced per top layer: the step scales it in one call
            tops = [l for l in range(s.L) if not s.feeds_next(l)]
            flat = torch.zeros(sum(s.shapes[l][0] * s.up_width[l] for l in tops), dtype=torch.float32,
                               device=s.device)
            out, o = [None] * s.L, 0
            for l in tops:
                m, n = s.shapes[l][0], s.up_width[l]
                out[l] = flat[o:o + m * n].view(m, n)
                o += m * n
            return out
        self.x_in = [[mk_x(l) for l in range(s.L)] for _ in range(2)]
        self.g_in = [mk_gs() for _ in range(2)]
        self.ready = [None, None]        # event: the set's copies have landed
        self.consumed = [None, None]     # event: the step that read the set has finished
        self.graphs = [None, None]
        self.fill, self.drain, self.pending = 0, 0, 0

    def submit(self, xs_host, gs_host):
        """Starts the copies of one batch (pinned host tensors, one per layer that takes input)."""
        assert self.pending < 2, "both staging sets are in use: call run() first"
        s, k = self.stack, self.fill
        cs = self.copy_stream
        if self.consumed[k] is not None:
            cs.wait_event(self.consumed[k])          # the step that read this set must be over
        with torch.cuda.stream(cs):
            for l in range(s.L):
                if self.x_in[k][l] is not None:
                    self.x_in[k][l][:, :s.shapes[l][1]].copy_(xs_host[l], non_blocking=True)
                if self.g_in[k][l] is not None:
                    self.g_in[k][l].copy_(gs_host[l], non_blocking=True)
            self.ready[k] = torch.cuda.Event()
            self.ready[k].record(cs)
        self.fill, self.pending = k ^ 1, self.pending + 1

    def run(self):
        """Runs the step on the oldest submitted batch and returns the device state after it."""
        assert self.pending > 0, "nothing submitted"
        s, k = self.stack, self.drain
        main = torch.cuda.current_stream()
        main.wait_event(self.ready[k])
        if self.use_graph and self.graphs[k] is None:
            s.step(self.x_in[k], self.g_in[k])       # this batch's step, call by call
            saved = s.graph
            self.graphs[k] = s.capture(self.x_in[k], self.g_in[k], warmup=0)   # recorded, not run
            s.graph = saved
        elif self.use_graph:
            self.graphs[k].replay()
        else:
            s.step(self.x_in[k], self.g_in[k])
        self.consumed[k] = torch.cuda.Event()
        self.consumed[k].record(main)
        self.drain, self.pending = k ^ 1, self.pending - 1
        return s.state.read()
