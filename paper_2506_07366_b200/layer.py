"""One MoE layer with prediction-driven expert duplication, driven through the C ABI.

`MoeLayer` owns the device buffers (allocated once with torch) and chains the six library calls on
the current stream; no step runs anywhere but in the library's kernels.
"""
from __future__ import annotations

import torch

from .binding import Context, Shape, workspace_bytes

# Row alignment of the slot buckets that the benchmark and the serving examples use: slot starts are
# multiples of 16 rows.  The grouped GEMM accepts any alignment (its tiles start at the slot's first
# row and only rows of the slot are written); a small one keeps the permuted buffers compact - with
# 288 slots, 128-row alignment would pad 32768 pairs to about 56000 rows, 16-row alignment to 35000.
ROW_ALIGN = 16


class MoeLayer:
    def __init__(self, shape: Shape, w_router, bias, w_gate, w_up, w_down, device=None):
        self.shape = s = shape
        self.ctx = Context(shape, device)
        dev = w_router.device
        self.w_router, self.bias = w_router, bias
        self.w_gate, self.w_up, self.w_down = w_gate, w_up, w_down
        i32 = dict(dtype=torch.int32, device=dev)
        bf = dict(dtype=torch.bfloat16, device=dev)
        self.x = torch.empty(s.T, s.D, **bf)             # staging for host inputs
        self.topk_idx = torch.empty(s.T, s.K, **i32)
        self.topk_w = torch.empty(s.T, s.K, dtype=torch.float32, device=dev)
        self.hist = torch.empty(s.E, **i32)
        self.replicas = torch.empty(s.E, **i32)
        self.slot_off = torch.empty(s.E + 1, **i32)
        self.slot_expert = torch.empty(s.S, **i32)
        self.bound = torch.empty(1, **i32)
        self.slot_row_off = torch.empty(s.S + 1, **i32)
        self.row_pair = torch.empty(s.Rcap, **i32)
        self.pair_row = torch.empty(s.T, s.K, **i32)
        self.xp = torch.empty(s.Rcap, s.D, **bf)
        self.h_ws = torch.empty(s.Rcap, s.F, **bf)
        self.yp = torch.empty(s.Rcap, s.D, **bf)
        self.out = torch.empty(s.T, s.D, **bf)
        self.workspace = torch.empty(max(16, workspace_bytes(s)), dtype=torch.uint8, device=dev)
        self.pred = torch.empty(s.E, **i32)
        self._planned = False

    def plan(self, predicted_hist, stream=None):
        """Replica plan from a predicted histogram (int32 [E], device or host tensor)."""
        self.pred.copy_(predicted_hist.to(torch.int32), non_blocking=True)
        self.ctx.plan(self.pred, self.shape.S, self.replicas, self.slot_off, self.slot_expert,
                      self.bound, stream)
        self._planned = True

    def forward(self, x, stream=None, out=None):
        """route (+ histogram + the counts dispatch ranks with: one kernel) -> dispatch (offsets, ranks,
        copies: one kernel) -> expert_ffn -> combine on device tensor x [T, D]: five launches.
        The result goes to `out` (bf16 [T, D]) if given, else to the layer's own buffer."""
        if not self._planned:
            raise RuntimeError("call plan(predicted_hist) before forward()")
        c = self.ctx
        out = self.out if out is None else out
        c.route_prepare(x, self.w_router, self.bias, self.topk_idx, self.topk_w, self.hist, self.workspace, stream)
        c.dispatch_prepared(x, self.topk_idx, self.hist, self.replicas, self.slot_off, self.slot_row_off,
                            self.row_pair, self.pair_row, self.xp, self.workspace, stream)
        c.expert_ffn(self.xp, self.slot_row_off, self.slot_expert, self.w_gate, self.w_up,
                     self.w_down, self.h_ws, self.yp, stream)
        c.combine(self.yp, self.pair_row, self.topk_w, out, stream)
        return out

    def start_prediction(self, replan_every: int = 1, ema_shift: int | None = None):
        """Distribution-Only Prediction in a loop (paper, Sections 3.1 and 3.2.1): from now on
        forward_predicted() feeds every batch's histogram to the predictor state and renews the
        plan from the prediction after every `replan_every`-th batch (the paper's prediction and
        placement frequency).  `ema_shift` = None keeps cumulative counts (every batch weighs the
        same); an integer k forgets old batches with weight 2^-k for the newest one.  The first
        batches run under the plan of an all-zero prediction (the spare slots spread evenly)."""
        if replan_every < 1:
            raise ValueError("replan_every >= 1")
        self._every, self._ema_shift, self._batches = int(replan_every), ema_shift, 0
        self._state = torch.zeros(self.shape.E, dtype=torch.int64, device=self.w_router.device)
        self.pred.zero_()
        self.ctx.plan(self.pred, self.shape.S, self.replicas, self.slot_off, self.slot_expert, self.bound)
        self._planned = True

    def forward_predicted(self, x, stream=None, out=None):
        """forward() under the current plan, then predictor update (and re-plan when due)."""
        out = self.forward(x, stream, out)
        if self._ema_shift is None:
            self.ctx.predictor_update(self.hist, self._state, self.pred, stream)
        else:
            self.ctx.predictor_update_ema(self.hist, self._state, self._ema_shift, self.pred, stream)
        self._batches += 1
        if self._batches % self._every == 0:
            self.ctx.plan(self.pred, self.shape.S, self.replicas, self.slot_off, self.slot_expert, self.bound,
                          stream)
        return out

    def capture(self, x, predicted_hist=None):
        """Records plan (if `predicted_hist`, an int32 [E] device tensor, is given) + forward on the
        fixed tensors `x` / `predicted_hist` into a CUDA graph and returns it; `graph.replay()` then
        runs the whole step with one launch, reading whatever those tensors hold at that moment and
        writing `self.out`.  Worth it for small, launch-bound batches (the 8 kernels of a tiny step
        take 0.12 ms launched one by one and 0.05 ms replayed).  The library's one-time set-up
        (tensor-map encoding, shared-memory opt-in) happens in the warm-up calls made here."""
        if predicted_hist is not None:
            self.pred.copy_(predicted_hist.to(torch.int32))
        elif not self._planned:
            raise RuntimeError("call plan(predicted_hist) first or pass predicted_hist")
        side = torch.cuda.Stream(x.device)
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()

        def step():
            if predicted_hist is not None:
                self.pred.copy_(predicted_hist, non_blocking=True)
                self.ctx.plan(self.pred, self.shape.S, self.replicas, self.slot_off, self.slot_expert, self.bound)
                self._planned = True
            self.forward(x)

        with torch.cuda.stream(side):
            for _ in range(2):
                step()
            with torch.cuda.graph(graph, stream=side):
                step()
        torch.cuda.current_stream().wait_stream(side)
        return graph

    def forward_host(self, x_host, out_host, stream=None):
        """Same, with (pinned) host tensors: copies x in, runs the layer, copies the result out."""
        self.x.copy_(x_host, non_blocking=True)
        out = self.forward(self.x, stream)
        out_host.copy_(out, non_blocking=True)
        return out_host


class HostPipeline:
    """Streams batches that live in pinned host memory through a MoeLayer.

    The host->device copy of batch i+1 and the device->host copy of result i-1 run on their own
    streams while batch i computes (PCIe is full duplex), with `depth` device buffers for inputs and
    results; events order every hand-over.  The layer's compute still runs on the current stream.
    """

    def __init__(self, layer: MoeLayer, depth: int = 2):
        s = layer.shape
        dev = layer.w_router.device
        self.layer, self.depth, self.n = layer, depth, 0
        bf = dict(dtype=torch.bfloat16, device=dev)
        self.x_dev = [torch.empty(s.T, s.D, **bf) for _ in range(depth)]
        self.out_dev = [torch.empty(s.T, s.D, **bf) for _ in range(depth)]
        self.s_in, self.s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        ev = lambda: [torch.cuda.Event() for _ in range(depth)]  # noqa: E731
        self.ev_in, self.ev_comp, self.ev_out = ev(), ev(), ev()

    def submit(self, x_host, out_host):
        """Queues one batch: x_host -> device -> layer -> out_host.  Returns immediately."""
        k = self.n % self.depth
        compute = torch.cuda.current_stream()
        reuse = self.n >= self.depth
        with torch.cuda.stream(self.s_in):
            if reuse:
                self.s_in.wait_event(self.ev_comp[k])      # the batch that used this input buffer is done
            else:
                self.s_in.wait_stream(compute)             # do not start before work already queued
            self.x_dev[k].copy_(x_host, non_blocking=True)
            self.ev_in[k].record(self.s_in)
        compute.wait_event(self.ev_in[k])
        if reuse:
            compute.wait_event(self.ev_out[k])             # the result buffer has been read out
        self.layer.forward(self.x_dev[k], out=self.out_dev[k])
        self.ev_comp[k].record(compute)
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(self.ev_comp[k])
            out_host.copy_(self.out_dev[k], non_blocking=True)
            self.ev_out[k].record(self.s_out)
        self.n += 1

    def drain(self):
        """Makes the current stream wait for every queued copy (call before timing/reading results)."""
        compute = torch.cuda.current_stream()
        compute.wait_stream(self.s_in)
        compute.wait_stream(self.s_out)
