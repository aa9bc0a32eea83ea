"""One pass of the whole FP8 hot path over a transformer block's tensors, as a sequence of C-ABI calls.

A step is: just-in-time quantize (amax -> scale -> cast; no transposed copies: the gradient products read the
row-major FP8 tensors in place) of every activation, weight
and upstream gradient; forward, dgrad and wgrad GEMMs of the QKV, output, up(-gate) and down projections;
quantize of Q, K, V, dO; FP8 attention forward and backward.  This module only owns device buffers (torch)
and the order of calls; every computation runs in the CUDA library.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

from . import binding as fp8
from . import synth

LAYERS = ("qkv", "o", "up", "down")


def _bits_to_dev(a: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(device).view(torch.bfloat16)


def _f32(device, v=0.0):
    return torch.full((1,), float(v), dtype=torch.float32, device=device)


@dataclass
class QTensor:
    """A BF16 tensor with its FP8 copy (and transposed copy) and the three device scalars of its scaling."""
    x: torch.Tensor
    fmt: int
    transpose: bool
    q: torch.Tensor = None
    qt: torch.Tensor = None
    amax: torch.Tensor = None
    scale: torch.Tensor = None
    scale_inv: torch.Tensor = None
    history: torch.Tensor = None       # delayed scaling: the last HISTORY_LEN abs-max values and the ring position
    head: torch.Tensor = None

    HISTORY_LEN = 1024                 # the length the paper trains with (Appendix E)

    def __post_init__(self):
        dev = self.x.device
        self.q = torch.empty(self.x.shape, dtype=torch.uint8, device=dev)
        if self.transpose:
            rows, cols = self.x.numel() // self.x.shape[-1], self.x.shape[-1]
            self.qt = torch.empty((cols, rows), dtype=torch.uint8, device=dev)
        self.amax, self.scale, self.scale_inv = _f32(dev), _f32(dev), _f32(dev)

    def quantize(self):
        fp8.fp8_quantize(self.x, self.fmt, self.q, self.qt, self.amax, self.scale, self.scale_inv)

    def quantize_delayed(self):
        """Delayed scaling (Appendix E): one pass casts under the scale of the history and records this step's
        abs-max; the history and the scale for the next step are updated afterwards.  The first call seeds the
        history with a just-in-time pass."""
        self.seed_history()
        # the scale computed after the previous step becomes this step's; this step's products read scale_inv, so the
        # update for the next step is written to the other pair of scalars
        (self.scale, self.scale_inv), self._next = self._next, (self.scale, self.scale_inv)
        fp8.fp8_cast(self.x, self.scale, self.fmt, self.q, self.qt, self.amax)
        fp8.fp8_scale_update(self.history, self.head, self.amax, self.fmt, 0, *self._next)

    def seed_history(self):
        """First call only: the history ring, and the first step's scale from a just-in-time amax pass."""
        if self.history is None:
            dev = self.x.device
            self.history = torch.zeros(self.HISTORY_LEN, dtype=torch.float32, device=dev)
            self.head = torch.zeros(1, dtype=torch.int32, device=dev)
            self._next = (_f32(dev), _f32(dev))
            fp8.fp8_amax(self.x, self.amax)
            fp8.fp8_scale_update(self.history, self.head, self.amax, self.fmt, 0, *self._next)

    @property
    def nbytes_in(self):
        return self.x.numel() * 2


def _share_scalars(*tensors):
    """Puts the (amax, scale, 1 / scale) scalars of several QTensors side by side in one buffer, the layout
    fp8_quantize_multi fills; every QTensor keeps its own one-element views."""
    buf = torch.zeros(3 * len(tensors), dtype=torch.float32, device=tensors[0].x.device)
    for i, t in enumerate(tensors):
        t.amax, t.scale, t.scale_inv = buf[3 * i:3 * i + 1], buf[3 * i + 1:3 * i + 2], buf[3 * i + 2:3 * i + 3]
    return buf


@dataclass
class Linear:
    name: str
    T: int
    N: int
    K: int
    x: QTensor
    w: QTensor
    dy: QTensor
    y: torch.Tensor = None
    dx: torch.Tensor = None
    dw: torch.Tensor = None
    scalars: torch.Tensor = None       # the nine scaling scalars of x, w, dy side by side

    @property
    def flops(self):            # forward + dgrad + wgrad
        return 3 * 2.0 * self.T * self.N * self.K


class BlockHotPath:
    """Device buffers of one block configuration and the step that runs the hot path over them."""

    KERNELS_PER_QUANTIZE = 2      # amax, cast (the cast derives the scale itself)
    KERNELS_PER_ATTN_BWD = 3    # prep, main, finish

    def __init__(self, cfg: synth.BlockConfig, device="cuda", with_linears=None, with_attention=True,
                 seq=None, batch=None, transposed_copies=False, attn_max_slack=0.0, scaling="jit", multi_quantize=True):
        # transposed_copies: also write [cols, rows] FP8 copies in the cast and run dgrad / wgrad on them (the
        # form a K-major-only tensor core needs); off by default, tcgen05 reads the operands in place
        # attn_max_slack: tau of the attention forward's reference maximum (0 = exact running maximum); P~ is then
        # scaled by 448 / 2^tau
        # scaling: "jit" = amax pass, scale, cast pass per tensor and step (fp8_quantize); "delayed" = one cast pass under
        # the scale of the abs-max history, which the pass itself feeds (Appendix E; the recipe the paper trains with)
        # multi_quantize: the just-in-time quantize of a group's tensors (x, w, dy of a projection; q, k, v, do) as one
        # reduction launch and one cast launch for the group (fp8_quantize_multi) instead of two launches per tensor:
        # the same codes and scales, fewer kernel boundaries; under delayed scaling the whole quantize of a group (casts,
        # amaxes, history updates, next scales) is one launch (fp8_quantize_delayed_multi)
        assert scaling in ("jit", "delayed")
        self.scaling = scaling
        self.multi_quantize = bool(multi_quantize)
        self.attn_max_slack = float(attn_max_slack)
        self.cfg = cfg
        self.device = torch.device(device)
        self.transposed_copies = transposed_copies
        self.with_linears = cfg.has_linears if with_linears is None else with_linears
        self.with_attention = with_attention
        self.B = cfg.batch if batch is None else batch
        self.N = cfg.seq if seq is None else seq
        self.linears: list[Linear] = []
        self.attn = None
        self.host_inputs: dict[str, np.ndarray] = {}
        self._delayed_sync = {}       # per group: the counter words of the one-launch delayed-scaling quantize
        self.gemm_events = []
        self.quant_events = []
        self.attn_events = []

    # ------------------------------------------------------------------ inputs
    def generate_host_inputs(self):
        """Seeded BF16 inputs on the host (numpy uint16 bits), keyed by tensor name."""
        h = {}
        if self.with_linears:
            for layer in LAYERS:
                x, w, dy = synth.linear_inputs(self.cfg, layer)
                h["x_" + layer], h["w_" + layer], h["dy_" + layer] = x, w, dy
        if self.with_attention:
            h["q"], h["k"], h["v"], h["do"] = synth.attention_inputs(self.cfg, seq=self.N, batch=self.B)
        self.host_inputs = h
        return h

    def allocate(self, host_inputs=None):
        h = self.host_inputs if host_inputs is None else host_inputs
        dev = self.device
        if self.with_linears:
            for layer in LAYERS:
                T, N, K = self.cfg.linear_shapes()[layer]
                lin = Linear(layer, T, N, K,
                             QTensor(_bits_to_dev(h["x_" + layer], dev), fp8.E4M3, self.transposed_copies),
                             QTensor(_bits_to_dev(h["w_" + layer], dev), fp8.E4M3, self.transposed_copies),
                             QTensor(_bits_to_dev(h["dy_" + layer], dev), fp8.E5M2, self.transposed_copies))
                lin.y = torch.empty((T, N), dtype=torch.bfloat16, device=dev)
                lin.dx = torch.empty((T, K), dtype=torch.bfloat16, device=dev)
                lin.dw = torch.empty((N, K), dtype=torch.bfloat16, device=dev)
                lin.scalars = _share_scalars(lin.x, lin.w, lin.dy)
                self.linears.append(lin)
        if self.with_attention:
            c = self.cfg
            a = {n: QTensor(_bits_to_dev(h[n], dev), fp8.E5M2 if n == "do" else fp8.E4M3, False)
                 for n in ("q", "k", "v", "do")}
            B, N, Hq, Hkv, d = self.B, self.N, c.n_q_heads, c.n_kv_heads, c.head_dim
            a["o"] = torch.empty((B, N, Hq, d), dtype=torch.bfloat16, device=dev)
            a["lse"] = torch.empty((B, Hq, N), dtype=torch.float32, device=dev)
            a["dq"] = torch.empty((B, N, Hq, d), dtype=torch.bfloat16, device=dev)
            a["dk"] = torch.empty((B, N, Hkv, d), dtype=torch.bfloat16, device=dev)
            a["dv"] = torch.empty((B, N, Hkv, d), dtype=torch.bfloat16, device=dev)
            a["ws"] = torch.empty(fp8.fp8_attention_workspace_bytes(1, B, N, Hq, Hkv, d), dtype=torch.uint8,
                                  device=dev)
            a["ds_scale"] = _f32(dev, 1.0)
            a["ds_amax"] = _f32(dev)
            a["softmax_scale"] = float(d) ** -0.5
            a["scalars"] = _share_scalars(a["q"], a["k"], a["v"], a["do"])
            self.attn = a
        return self

    def input_tensors(self):
        """(name, device BF16 tensor) of every input of a step, in a fixed order."""
        out = []
        for lin in self.linears:
            out += [("x_" + lin.name, lin.x.x), ("w_" + lin.name, lin.w.x), ("dy_" + lin.name, lin.dy.x)]
        if self.attn is not None:
            out += [(n, self.attn[n].x) for n in ("q", "k", "v", "do")]
        return out

    def output_tensors(self):
        out = []
        for lin in self.linears:
            out += [("y_" + lin.name, lin.y), ("dx_" + lin.name, lin.dx), ("dw_" + lin.name, lin.dw)]
        if self.attn is not None:
            out += [(n, self.attn[n]) for n in ("o", "lse", "dq", "dk", "dv")]
        return out

    # ------------------------------------------------------------------ host-to-host step
    def step_host(self, h_in: dict, h_out: dict, wait: bool = True):
        """One step on pinned host buffers: inputs go up, every output comes back.

        Three streams: uploads, the kernels (the caller's current stream), downloads.  The copy engines run both
        directions at once and under the kernels, so a step costs about max(upload, download) instead of their
        sum.  h_in / h_out map the names of input_tensors() / output_tensors() to pinned host tensors.  With
        ``wait`` the current stream has waited for the last download on return.  Without it consecutive steps
        overlap as well (the uploads of one step run while the previous step's outputs are still going down; a
        group's kernels wait only for the previous download of their own outputs): call ``finish_host()`` before
        reading the host buffers.
        """
        main = torch.cuda.current_stream(self.device)
        if not hasattr(self, "_up"):
            self._up, self._down = torch.cuda.Stream(self.device), torch.cuda.Stream(self.device)
            self._downloaded = None
        up, down = self._up, self._down
        up.wait_stream(main)          # the previous step's kernels have read the device inputs
        groups = []                   # (inputs, kernels, outputs) per independent piece of the step
        for lin in self.linears:
            ins = [("x_" + lin.name, lin.x.x), ("w_" + lin.name, lin.w.x), ("dy_" + lin.name, lin.dy.x)]
            outs = [("y_" + lin.name, lin.y), ("dx_" + lin.name, lin.dx), ("dw_" + lin.name, lin.dw)]
            groups.append((ins, lambda lin=lin: self._run_linear(lin), outs))
        if self.attn is not None:
            a = self.attn
            ins = [(n, a[n].x) for n in ("q", "k", "v", "do")]
            outs = [(n, a[n]) for n in ("o", "lse", "dq", "dk", "dv")]
            groups.append((ins, self._run_attention, outs))
        ready = []
        with torch.cuda.stream(up):
            for ins, _, _ in groups:
                for name, d in ins:
                    d.copy_(h_in[name], non_blocking=True)
                e = torch.cuda.Event()
                e.record(up)
                ready.append(e)
        prev, downloaded = self._downloaded, []
        for g, ((ins, run, outs), e) in enumerate(zip(groups, ready)):
            main.wait_event(e)
            if prev is not None:
                main.wait_event(prev[g])          # the previous step's copy of these outputs has left the device
            run()
            done = torch.cuda.Event()
            done.record(main)
            with torch.cuda.stream(down):
                down.wait_event(done)
                for name, d in outs:
                    h_out[name].copy_(d, non_blocking=True)
                gone = torch.cuda.Event()
                gone.record(down)
            downloaded.append(gone)
        self._downloaded = downloaded
        if wait:
            self.finish_host()

    def finish_host(self):
        """The current stream waits for every download issued by step_host()."""
        if hasattr(self, "_down"):
            torch.cuda.current_stream(self.device).wait_stream(self._down)
            self._downloaded = None

    def step_host_abi(self, h_in: dict, h_out: dict):
        """The same step through the host-buffer entry points of the C ABI: one fp8_linear_step_host per projection
        and one fp8_attention_step_host, each on a device workspace of its own, so that the library overlaps the
        copies of one group with the kernels of another.  Returns once enqueued; ``fp8.fp8_host_sync()`` before
        reading h_out.  dS is quantised with the scale this object holds at the first call (a host value)."""
        if not hasattr(self, "_host_ws"):
            ws = {}
            for lin in self.linears:
                ws[lin.name] = torch.empty(fp8.fp8_linear_step_host_workspace_bytes(lin.T, lin.N, lin.K),
                                           dtype=torch.uint8, device=self.device)
            if self.attn is not None:
                c = self.cfg
                ws["attn"] = torch.empty(fp8.fp8_attention_step_host_workspace_bytes(
                    self.B, self.N, c.n_q_heads, c.n_kv_heads, c.head_dim), dtype=torch.uint8, device=self.device)
                self._host_ds_scale = float(self.attn["ds_scale"].item())
            self._host_ws = ws
        for lin in self.linears:
            n = lin.name
            fp8.fp8_linear_step_host(h_in["x_" + n], h_in["w_" + n], h_in["dy_" + n], h_out["y_" + n], h_out["dx_" + n],
                                     h_out["dw_" + n], self._host_ws[n])
        if self.attn is not None:
            fp8.fp8_attention_step_host(h_in["q"], h_in["k"], h_in["v"], h_in["do"], self.attn["softmax_scale"],
                                        self._host_ds_scale, True, h_out["o"], h_out["lse"], h_out["dq"], h_out["dk"],
                                        h_out["dv"], self._host_ws["attn"])

    def _quantize_group(self, tensors, scalars):
        """Quantize of the tensors of one group under the configured recipe."""
        if self.scaling == "delayed" and self.multi_quantize and not self.transposed_copies:
            # one launch for the group: casts under the scales the previous step left in _next[0] (published to scale /
            # scale_inv for the products), amaxes, history updates, and the next step's scales back into _next[0]; the same
            # pointers every step
            for t in tensors:
                t.seed_history()
            key = id(tensors[0])
            if key not in self._delayed_sync:
                self._delayed_sync[key] = torch.zeros(2 * len(tensors), dtype=torch.int32, device=self.device)
            fp8.fp8_quantize_delayed_multi([t.x for t in tensors], [t.fmt for t in tensors], [t.q for t in tensors],
                                           [t.history for t in tensors], [t.head for t in tensors],
                                           [t._next[0] for t in tensors], [t.amax for t in tensors],
                                           [t.scale for t in tensors], [t.scale_inv for t in tensors], 0,
                                           self._delayed_sync[key])
        elif self.scaling == "delayed":
            for t in tensors:
                t.quantize_delayed()
        elif self.multi_quantize and not self.transposed_copies:
            fp8.fp8_quantize_multi([t.x for t in tensors], [t.fmt for t in tensors], [t.q for t in tensors], scalars)
        else:
            for t in tensors:
                t.quantize()

    def _run_linear(self, lin):
        self._quantize_group((lin.x, lin.w, lin.dy), lin.scalars)
        fp8.fp8_linear_fwd(lin.x.q, lin.w.q, lin.x.scale_inv, lin.w.scale_inv, lin.y)
        if self.transposed_copies:
            fp8.fp8_linear_dgrad(lin.dy.q, lin.w.qt, lin.dy.scale_inv, lin.w.scale_inv, lin.dx)
            fp8.fp8_linear_wgrad(lin.dy.qt, lin.x.qt, lin.dy.scale_inv, lin.x.scale_inv, lin.dw)
        else:
            fp8.fp8_linear_dgrad_rm(lin.dy.q, lin.w.q, lin.dy.scale_inv, lin.w.scale_inv, lin.dx)
            fp8.fp8_linear_wgrad_rm(lin.dy.q, lin.x.q, lin.dy.scale_inv, lin.x.scale_inv, lin.dw)

    def _run_attention(self):
        a = self.attn
        self._quantize_group([a[n] for n in ("q", "k", "v", "do")], a["scalars"])
        fp8.fp8_attention_fwd(a["q"].q, a["k"].q, a["v"].q, a["q"].scale_inv, a["k"].scale_inv, a["v"].scale_inv,
                              a["softmax_scale"], True, a["o"], a["lse"], None,
                              p_scale=448.0 / 2.0 ** self.attn_max_slack, max_slack=self.attn_max_slack)
        fp8.fp8_attention_bwd(a["q"].q, a["k"].q, a["v"].q, a["do"].q, a["o"], a["lse"], a["q"].scale_inv,
                              a["k"].scale_inv, a["v"].scale_inv, a["do"].scale_inv, a["softmax_scale"],
                              a["ds_scale"], True, a["dq"], a["dk"], a["dv"], a["ws"], ds_amax=a["ds_amax"])

    # ------------------------------------------------------------------ work accounting
    def gemm_flops(self):
        return sum(l.flops for l in self.linears)

    def attention_flops(self):
        """Causal attention: forward 2*B*Hq*N^2*d (half of the dense 4*N^2*d), backward 2.5x that."""
        if self.attn is None:
            return 0.0
        c = self.cfg
        fwd = 2.0 * self.B * c.n_q_heads * self.N * self.N * c.head_dim
        return 3.5 * fwd

    def quantize_bytes(self):
        """Algorithmic HBM bytes of the JIT quantize calls: 2 (amax read) + 2 (cast read) + 1 per FP8 copy."""
        b = 0
        rd = 4 if self.scaling == "jit" else 2          # BF16 read twice (amax pass, cast pass) or once
        for lin in self.linears:
            for t in (lin.x, lin.w, lin.dy):
                b += t.x.numel() * (rd + 1 + (1 if t.transpose else 0))
        if self.attn is not None:
            for n in ("q", "k", "v", "do"):
                b += self.attn[n].x.numel() * (rd + 1)
        return b

    def launches_per_step(self):
        n = 0
        kq = self.KERNELS_PER_QUANTIZE         # delayed scaling: cast (+amax) and the history update, also two
        grouped = self.multi_quantize and not self.transposed_copies
        # per group: one reduction + one cast (just-in-time) or one launch (delayed); else two launches per tensor
        kg = 1 if self.scaling == "delayed" else kq
        for _ in self.linears:
            n += (kg if grouped else 3 * kq) + 3
        if self.attn is not None:
            n += (kg if grouped else 4 * kq) + 1 + self.KERNELS_PER_ATTN_BWD
        return n

    # ------------------------------------------------------------------ the step
    def calibrate_ds_scale(self):
        """Delayed-scaling style: one backward with scale 1 gives amax(dS); scale = 57344 / amax."""
        if self.attn is None:
            return
        a = self.attn
        a["ds_scale"].fill_(1.0)
        self.step()
        tmp_scale_inv = _f32(self.device)
        fp8.fp8_scale(a["ds_amax"], fp8.E5M2, 0, a["ds_scale"], tmp_scale_inv)
        torch.cuda.synchronize(self.device)

    def capture_graph(self):
        """Captures one step (the same launches) into a CUDA graph and returns it; ``graph.replay()`` then runs the
        step with one submission.  The step makes no host synchronisation, so it is capturable as it is.  Worth it
        where the step is launch-bound (small configurations); the large ones are bound by the kernels.  Delayed
        scaling is capturable in its one-launch form (the same pointers every step); the per-tensor form alternates
        between two pairs of scale scalars on the host, which one captured step cannot express."""
        if self.scaling != "jit" and not (self.multi_quantize and not self.transposed_copies):
            raise ValueError("capture_graph: the per-tensor delayed-scaling step alternates its scale buffers between "
                             "steps on the host; capture needs scaling='jit' or the one-launch group quantize")
        side = torch.cuda.Stream(self.device)
        side.wait_stream(torch.cuda.current_stream(self.device))
        with torch.cuda.stream(side):
            self.step()                       # every lazy initialisation happens outside the capture
        torch.cuda.current_stream(self.device).wait_stream(side)
        torch.cuda.synchronize(self.device)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.step()
        return graph

    def step_overlapped(self, time_gemms: bool = False):
        """The launches of step() on two streams: every quantize call goes to a side stream, the products and the
        attention stay on the current one and wait (events) only for the operands they read.  The quantize passes are
        HBM-bound and their CTAs fit beside the persistent GEMM CTAs of an SM, so they run in the shadow of the
        products of the groups before them; only the first group's quantize is exposed.  Same kernels, same bits."""
        main = torch.cuda.current_stream(self.device)
        if getattr(self, "_qstream", None) is None:
            self._qstream = torch.cuda.Stream(self.device)
        side = self._qstream
        side.wait_stream(main)              # the previous step's products have read the FP8 buffers about to be rewritten
        ready = []
        with torch.cuda.stream(side):
            for lin in self.linears:
                self._quantize_group((lin.x, lin.w, lin.dy), lin.scalars)
                ev = torch.cuda.Event()
                ev.record(side)
                ready.append(ev)
            if self.attn is not None:
                self._quantize_group([self.attn[n] for n in ("q", "k", "v", "do")], self.attn["scalars"])
                ev = torch.cuda.Event()
                ev.record(side)
                ready.append(ev)
        gev = []

        def gemm(fn, *args):
            if time_gemms:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                fn(*args)
                e1.record()
                gev.append((e0, e1))
            else:
                fn(*args)

        for lin, ev in zip(self.linears, ready):
            main.wait_event(ev)
            gemm(fp8.fp8_linear_fwd, lin.x.q, lin.w.q, lin.x.scale_inv, lin.w.scale_inv, lin.y)
            if self.transposed_copies:
                gemm(fp8.fp8_linear_dgrad, lin.dy.q, lin.w.qt, lin.dy.scale_inv, lin.w.scale_inv, lin.dx)
                gemm(fp8.fp8_linear_wgrad, lin.dy.qt, lin.x.qt, lin.dy.scale_inv, lin.x.scale_inv, lin.dw)
            else:
                gemm(fp8.fp8_linear_dgrad_rm, lin.dy.q, lin.w.q, lin.dy.scale_inv, lin.w.scale_inv, lin.dx)
                gemm(fp8.fp8_linear_wgrad_rm, lin.dy.q, lin.x.q, lin.dy.scale_inv, lin.x.scale_inv, lin.dw)
        if time_gemms:
            self.gemm_events.append(gev)
        if self.attn is not None:
            a = self.attn
            main.wait_event(ready[-1])
            fp8.fp8_attention_fwd(a["q"].q, a["k"].q, a["v"].q, a["q"].scale_inv, a["k"].scale_inv, a["v"].scale_inv,
                                  a["softmax_scale"], True, a["o"], a["lse"], None,
                                  p_scale=448.0 / 2.0 ** self.attn_max_slack, max_slack=self.attn_max_slack)
            fp8.fp8_attention_bwd(a["q"].q, a["k"].q, a["v"].q, a["do"].q, a["o"], a["lse"], a["q"].scale_inv,
                                  a["k"].scale_inv, a["v"].scale_inv, a["do"].scale_inv, a["softmax_scale"],
                                  a["ds_scale"], True, a["dq"], a["dk"], a["dv"], a["ws"], ds_amax=a["ds_amax"])

    def step(self, time_gemms: bool = False):
        """One pass of the hot path.  With ``time_gemms`` every GEMM launch, every quantize group and the two attention
        calls are bracketed by CUDA events on the launching stream (appended to gemm_events / quant_events /
        attn_events, one list per step)."""
        ev, qev, aev = [], [], []

        def timed(dst, fn, *args, **kw):
            if time_gemms:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                fn(*args, **kw)
                e1.record()
                dst.append((e0, e1))
            else:
                fn(*args, **kw)

        def gemm(fn, *args, **kw):
            timed(ev, fn, *args, **kw)

        for lin in self.linears:
            timed(qev, self._quantize_group, (lin.x, lin.w, lin.dy), lin.scalars)
            gemm(fp8.fp8_linear_fwd, lin.x.q, lin.w.q, lin.x.scale_inv, lin.w.scale_inv, lin.y)
            if self.transposed_copies:
                gemm(fp8.fp8_linear_dgrad, lin.dy.q, lin.w.qt, lin.dy.scale_inv, lin.w.scale_inv, lin.dx)
                gemm(fp8.fp8_linear_wgrad, lin.dy.qt, lin.x.qt, lin.dy.scale_inv, lin.x.scale_inv, lin.dw)
            else:
                gemm(fp8.fp8_linear_dgrad_rm, lin.dy.q, lin.w.q, lin.dy.scale_inv, lin.w.scale_inv, lin.dx)
                gemm(fp8.fp8_linear_wgrad_rm, lin.dy.q, lin.x.q, lin.dy.scale_inv, lin.x.scale_inv, lin.dw)
        if self.attn is not None:
            a = self.attn
            timed(qev, self._quantize_group, [a[n] for n in ("q", "k", "v", "do")], a["scalars"])
            timed(aev, fp8.fp8_attention_fwd, a["q"].q, a["k"].q, a["v"].q, a["q"].scale_inv, a["k"].scale_inv,
                  a["v"].scale_inv, a["softmax_scale"], True, a["o"], a["lse"], None,
                  p_scale=448.0 / 2.0 ** self.attn_max_slack, max_slack=self.attn_max_slack)
            timed(aev, fp8.fp8_attention_bwd, a["q"].q, a["k"].q, a["v"].q, a["do"].q, a["o"], a["lse"],
                  a["q"].scale_inv, a["k"].scale_inv, a["v"].scale_inv, a["do"].scale_inv, a["softmax_scale"],
                  a["ds_scale"], True, a["dq"], a["dk"], a["dv"], a["ws"], ds_amax=a["ds_amax"])
        if time_gemms:
            self.gemm_events.append(ev)
            self.quant_events.append(qev)
            self.attn_events.append(aev)
