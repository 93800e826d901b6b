"""Host-side schedule of the ShadowSync hot path on one GPU (Algorithm 1).

R trainer replicas live on the device as separate buffers.  Each replica owns CUDA streams above the
shadow stream's priority on which its training step is enqueued (four library calls: embedding forward,
MLP forward, MLP backward + dense Adagrad, embedding backward + row-wise Adagrad; the MLP calls on the
highest priority, the embedding calls one level below where the device has the levels).  The shadow thread of the
paper (Section 3.2) is a host thread that keeps enqueuing one synchronisation kernel after another
on a separate lowest-priority stream; it shares no event or dependency with the training streams.

This module allocates torch tensors and calls the binding; it computes nothing itself.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as ss


class DeviceBatch:
    """One batch resident on the device.  The four arrays are views of ONE device buffer (`storage`, each array on a
    256-byte boundary), so a batch staged on the host in the same layout (`pack_host`) arrives with a single copy."""

    FIELDS = (("indices", torch.int32), ("offsets", torch.int32), ("dense", torch.float32), ("labels", torch.float32))

    @staticmethod
    def _layout(arrays):
        offs, o = [], 0
        for a in arrays:
            offs.append(o)
            o += (a.numel() * a.element_size() + 255) // 256 * 256
        return offs, o

    @classmethod
    def _as_tensors(cls, indices, offsets, dense, labels):
        out = []
        for a, (_, dt) in zip((indices, offsets, dense, labels), cls.FIELDS):
            t = a if isinstance(a, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(a))
            out.append(t.to(dtype=dt).contiguous())
        return out

    @classmethod
    def pack_host(cls, indices, offsets, dense, labels):
        """The batch in the layout of `storage`, in pinned host memory."""
        ts = cls._as_tensors(indices, offsets, dense, labels)
        offs, total = cls._layout(ts)
        buf = torch.zeros(total, dtype=torch.uint8).pin_memory()
        for t, o in zip(ts, offs):
            n = t.numel() * t.element_size()
            buf[o:o + n] = t.cpu().reshape(-1).view(torch.uint8)
        return buf

    def __init__(self, indices, offsets, dense, labels, device="cuda"):
        ts = self._as_tensors(indices, offsets, dense, labels)
        offs, total = self._layout(ts)
        self.storage = torch.zeros(total, dtype=torch.uint8, device=device)
        for t, o, (name, dt) in zip(ts, offs, self.FIELDS):
            n = t.numel() * t.element_size()
            view = self.storage[o:o + n].view(dt).view(t.shape)
            view.copy_(t.to(device=device, non_blocking=True) if t.device != view.device else t)
            setattr(self, name, view)
        self.L = int(self.indices.numel())


class Replica:
    """Buffers of one trainer replica: w^(i), its Adagrad accumulator, bf16 mirror, activations, stream."""

    def __init__(self, model: "Model", w0_flat: torch.Tensor, priority: int, max_L: int, keep_sort_outputs: bool,
                 share: Optional["Replica"] = None):
        m, dev = model, model.device
        B, spec = m.B, m.spec
        if share is not None:
            # a further worker of the same trainer: its own activations and streams, but the trainer's single
            # copy of the parameters and of the optimizer state, updated lock-free (Section 3.2)
            self.w, self.acc, self.w_bf16 = share.w, share.acc, share.w_bf16
        else:
            self.w = w0_flat.clone()
            self.acc = torch.zeros_like(self.w)
            self.w_bf16 = torch.empty(spec.param_count, dtype=torch.bfloat16, device=dev) if spec.bf16 else None
            if spec.bf16:
                ss.ss_to_bf16(self.w, self.w_bf16, spec.param_count)
        self.concat_f32 = torch.zeros(B, spec.W, dtype=torch.float32, device=dev) if (not spec.bf16 or m.keep_f32_concat) else None
        self.concat_bf16 = torch.zeros(B, spec.W, dtype=torch.bfloat16, device=dev) if spec.bf16 else None
        self.logit = torch.empty(B, dtype=torch.float32, device=dev)
        self.prob = torch.empty(B, dtype=torch.float32, device=dev)
        self.loss = torch.zeros(1, dtype=torch.float32, device=dev)
        self.grad_pooled = torch.empty(B, m.T * m.D, dtype=torch.float32, device=dev)
        self.mlp_ws = torch.empty(ss.ss_mlp_workspace_bytes(spec, B), dtype=torch.uint8, device=dev)
        self.emb_ws = torch.empty(ss.ss_embbag_bwd_workspace_bytes(m.T, m.N, m.D, B, max_L), dtype=torch.uint8, device=dev)
        self.num_unique = torch.zeros(1, dtype=torch.int32, device=dev)
        self.uniq_keys = self.seg_off = self.perm = None
        if keep_sort_outputs:
            self.uniq_keys = torch.empty(max_L, dtype=torch.int32, device=dev)
            self.seg_off = torch.empty(max_L + 1, dtype=torch.int32, device=dev)
            self.perm = torch.empty(max_L, dtype=torch.int32, device=dev)
        # The embedding calls are long kernels that fill the device and are bound by memory throughput; the MLP
        # calls are chains of short kernels bound by latency.  The MLP chain therefore gets the highest priority
        # and the embedding calls a level in between (still above the shadow stream): blocks of an MLP kernel
        # are placed as soon as a slot frees up instead of queueing behind another replica's gather.
        self.stream = torch.cuda.Stream(device=dev, priority=model.prio_embedding)
        # the index sort of the backward runs here: one block per table on few SMs, and the reduction waits for it,
        # so it goes in between where the device has a level left (measured +2 % examples/s)
        self.side = torch.cuda.Stream(device=dev, priority=model.prio_sort)
        self.mlp = torch.cuda.Stream(device=dev, priority=priority)
        self.steps_done = 0


class Model:
    """Shared embedding tables h, R replicas of the dense parameters, and the centre/global copy."""

    def __init__(self, T: int, N: int, D: int, B: int, bottom: Sequence[int], top: Sequence[int], bf16: bool,
                 R: int, w0_flat: torch.Tensor, tables: torch.Tensor, lr: float = 0.01, eps: float = 1e-8,
                 max_L: int = 0, keep_sort_outputs: bool = False, keep_f32_concat: bool = False, device="cuda",
                 workers: int = 1):
        self.T, self.N, self.D, self.B, self.R = T, N, D, B, R
        self.lr, self.eps = lr, eps
        self.device = device
        self.keep_f32_concat = keep_f32_concat
        self.spec = ss.MlpSpec(bottom, top, bf16)
        assert self.spec.W == (1 + T) * D and self.spec.D0 == D, "concat = [bottom_out | T pooled vectors]"
        assert w0_flat.numel() == self.spec.param_count
        self.tables = tables                       # float32 [T, N, D]
        self.row_state = torch.zeros(T * N, dtype=torch.float32, device=device)
        self.d_status = torch.zeros(1, dtype=torch.int32, device=device)
        lo, hi = torch.cuda.Stream.priority_range()   # (lowest priority value, highest), e.g. (0, -5)
        self.prio_low, self.prio_high = lo, hi
        self.prio_embedding = hi + min(2, max(0, (lo - hi) - 1))   # between the two when the device has the levels
        # only while the sort is the light per-table kernel: the tiled passes of larger batches fill the device and,
        # given precedence over the other replicas' embedding calls, cost a quarter of the throughput (measured)
        # ... and while the sorts of all replicas together (one SM per table each) leave SMs free: with R*T beyond the
        # SM count the raised level costs 2 % instead of gaining 2 % (measured at R=8, T=26)
        light_sort = 0 < max_L <= T * ss.SS_TABLE_SORT_CAP and R * workers * T <= ss.ss_num_sms()
        self.prio_sort = self.prio_embedding - 1 if (light_sort and self.prio_embedding - 1 > hi) else self.prio_embedding
        self.replicas: List[Replica] = [Replica(self, w0_flat, hi, max_L, keep_sort_outputs) for _ in range(R)]
        # workers[r][k]: worker k of trainer r; worker 0 is the replica itself, further workers share its parameters
        # (the paper's intra-trainer Hogwild: m threads, each on its own batch, updating one local copy)
        self.workers: List[List[Replica]] = [
            [rep] + [Replica(self, w0_flat, hi, max_L, keep_sort_outputs, share=rep) for _ in range(workers - 1)]
            for rep in self.replicas]
        self.center = w0_flat.clone()              # w^PS (EASGD) / w^global (MA, BMUF), initialised to w0
        self.delta = torch.zeros_like(self.center)  # BMUF block momentum
        self.sync_stream = torch.cuda.Stream(device=device, priority=lo)
        torch.cuda.synchronize()

    # ---------------------------------------------------------------- training step of one replica
    def step(self, r: int, batch: DeviceBatch, stream: Optional[torch.cuda.Stream] = None,
             overlap_sort: bool = True, worker: int = 0) -> None:
        """Enqueue one worker iteration of Algorithm 1 for replica r on its stream (no synchronisation).

        With overlap_sort the sort / unique half of the embedding backward, which needs only the batch's
        indices, is forked onto the replica's side stream at the start of the step and joined before the
        gradient reduction, so it runs under the forward and backward passes of the MLP.
        """
        rep, sp = self.workers[r][worker], self.spec
        s = stream or rep.stream
        T, N, D, B = self.T, self.N, self.D, self.B
        if overlap_sort:
            fork = torch.cuda.Event()
            fork.record(s)
            rep.side.wait_event(fork)
            ss.ss_embbag_bwd_sort(T, N, D, batch.indices, batch.offsets, B, batch.L, rep.emb_ws, rep.uniq_keys,
                                  rep.seg_off, rep.perm, rep.num_unique, self.d_status, rep.side)
            join = torch.cuda.Event()
            join.record(rep.side)
        ss.ss_embbag_fwd(self.tables, T, N, D, batch.indices, batch.offsets, B, rep.concat_f32, sp.W,
                         rep.concat_bf16, sp.W, D, self.d_status, s)
        # on the replica's own stream the MLP calls move to its high-priority stream (a caller's stream is kept)
        m = rep.mlp if s is rep.stream else s
        if m is not s:
            e = torch.cuda.Event()
            e.record(s)
            m.wait_event(e)
        ss.ss_mlp_fwd(sp, rep.w, rep.w_bf16, batch.dense, rep.concat_f32, rep.concat_bf16, B, batch.labels,
                      rep.logit, rep.prob, rep.loss, rep.mlp_ws, m)
        ss.ss_mlp_bwd(sp, rep.w, rep.w_bf16, rep.acc, None, batch.dense, rep.concat_f32, rep.concat_bf16,
                      batch.labels, rep.prob, B, self.lr, self.eps, 1, rep.grad_pooled, T * D, rep.mlp_ws, m)
        if m is not s:
            e = torch.cuda.Event()
            e.record(m)
            s.wait_event(e)
        if overlap_sort:
            s.wait_event(join)
            ss.ss_embbag_bwd_apply(self.tables, self.row_state, T, N, D, B, batch.L, rep.grad_pooled, T * D, 0,
                                   self.lr, self.eps, rep.emb_ws, self.d_status, s)
        else:
            ss.ss_embbag_bwd_adagrad(self.tables, self.row_state, T, N, D, batch.indices, batch.offsets, B, batch.L,
                                     rep.grad_pooled, T * D, 0, self.lr, self.eps, rep.emb_ws, rep.uniq_keys,
                                     rep.seg_off, rep.perm, rep.num_unique, self.d_status, s)
        rep.steps_done += 1

    # ---------------------------------------------------------------- one synchronisation pass
    def sync(self, rule: str, alpha: float, eta: float = 1.0, mu: float = 0.0, stream=None, flags: int = 0) -> None:
        """Enqueue one pass of Algorithm 2 ("easgd"), 3 ("ma") or 4 ("bmuf") over all replicas."""
        s = stream or self.sync_stream
        ws = [rep.w for rep in self.replicas]
        mirrors = [rep.w_bf16 for rep in self.replicas] if self.spec.bf16 else None
        n = self.spec.param_count
        if rule == "easgd":
            ss.ss_sync_easgd(ws, self.center, n, alpha, flags, mirrors, s)
        elif rule == "ma":
            ss.ss_sync_ma(ws, self.center, n, alpha, flags, mirrors, s)
        elif rule == "bmuf":
            ss.ss_sync_bmuf(ws, self.center, self.delta, n, alpha, eta, mu, flags, mirrors, s)
        else:
            raise ValueError(rule)

    def foreground_sync(self, rule: str, alpha: float, eta: float = 1.0, mu: float = 0.0, flags: int = 0) -> None:
        """The foreground variants the paper compares against (FR-EASGD, FR-MA, FR-BMUF; Section 4): the
        same kernels, but enqueued on the training streams, so training waits for them.

        EASGD is centralised: every replica interpolates with the centre on its own, on its own stream, as
        a worker would with the sync PS (replicas' passes may interleave; the centre is shared lock-free).
        MA and BMUF need all replicas: every training stream joins, one pass runs, every stream waits for it.
        """
        n = self.spec.param_count
        if rule == "easgd":
            for rep in self.replicas:
                ss.ss_sync_easgd([rep.w], self.center, n, alpha, flags, [rep.w_bf16] if self.spec.bf16 else None,
                                 rep.stream)
            return
        lead = self.replicas[0].stream
        for rep in self.replicas[1:]:
            e = torch.cuda.Event()
            e.record(rep.stream)
            lead.wait_event(e)
        self.sync(rule, alpha, eta, mu, stream=lead, flags=flags)
        done = torch.cuda.Event()
        done.record(lead)
        for rep in self.replicas[1:]:
            rep.stream.wait_event(done)

    def status(self) -> int:
        """Device-detected problems so far: the SS_DEV_* bits of malformed input in the low byte, and from bit 8
        up the code of a tensor-core kernel's bounded wait that ran out (0 = none).  Synchronises the device."""
        return int(self.d_status.item()) | (ss.ss_device_error(False) << 8)


class ShadowLoop:
    """The shadow thread: loops the synchronisation on the low-priority stream, unaware of training.

    The loop itself is a native host thread inside the library (ss_shadow_start), so it neither holds nor
    waits for the Python interpreter lock.  At most `max_in_flight` sync kernels are queued ahead of the
    device; `pause_s` > 0 paces the loop.
    """

    def __init__(self, model: Model, rule: str, alpha: float, eta: float = 1.0, mu: float = 0.0,
                 max_in_flight: int = 2, pause_s: float = 0.0, max_rounds: int = 1 << 40):
        self.model, self.rule, self.alpha, self.eta, self.mu = model, rule, alpha, eta, mu
        self.max_in_flight, self.pause_s, self.max_rounds = max_in_flight, pause_s, max_rounds
        self._handle = None
        self._final = 0

    @property
    def rounds(self) -> int:
        return ss.ss_shadow_rounds(self._handle) if self._handle is not None else self._final

    def start(self) -> "ShadowLoop":
        m = self.model
        ws = [rep.w for rep in m.replicas]
        mirrors = [rep.w_bf16 for rep in m.replicas] if m.spec.bf16 else None
        self._handle = ss.ss_shadow_start(self.rule, ws, m.center, m.delta, m.spec.param_count, self.alpha, self.eta,
                                          self.mu, 0, mirrors, m.sync_stream, self.max_in_flight,
                                          int(self.pause_s * 1e6), self.max_rounds)
        return self

    def pause(self) -> int:
        """Stop enqueuing, wait for the queued passes; returns the number of passes completed so far."""
        ss.ss_shadow_pause(self._handle, True)
        return self.rounds

    def resume(self) -> None:
        ss.ss_shadow_pause(self._handle, False)

    def stop(self) -> int:
        if self._handle is not None:
            self._final = ss.ss_shadow_stop(self._handle)
            self._handle = None
        return self._final


# ------------------------------------------------------------------------------------------
def pack_params(spec: ss.MlpSpec, layers) -> np.ndarray:
    """Per-layer (W [out,in], b [out]) float32 arrays -> the flat padded vector of the library's layout."""
    flat = np.zeros(spec.param_count, dtype=np.float32)
    for l, (W, b) in enumerate(layers):
        fin, fout = spec.layer_dims[l]
        assert W.shape == (fout, fin) and b.shape == (fout,)
        flat[spec.w_off[l]: spec.w_off[l] + fin * fout] = W.ravel()
        flat[spec.b_off[l]: spec.b_off[l] + fout] = b
    return flat


def unpack_params(spec: ss.MlpSpec, flat: np.ndarray):
    out = []
    for l, (fin, fout) in enumerate(spec.layer_dims):
        W = flat[spec.w_off[l]: spec.w_off[l] + fin * fout].reshape(fout, fin).copy()
        b = flat[spec.b_off[l]: spec.b_off[l] + fout].copy()
        out.append((W, b))
    return out


def device_tables(cfg, device="cuda") -> torch.Tensor:
    """Fill the synthetic tables of a workload configuration on the device: float32 [T, N, D]."""
    from . import synth
    t = torch.empty(cfg.T, cfg.N, cfg.D, dtype=torch.float32, device=device)
    ss.ssh_fill_uniform(t, t.numel(), int(synth.table_key(cfg)), 0, float(np.float32(synth.TABLE_HI - synth.TABLE_LO)),
                        float(np.float32(0.5 * (synth.TABLE_HI + synth.TABLE_LO))))
    return t
