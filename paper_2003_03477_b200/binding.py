"""ctypes binding of libshadowsync.so: argument marshalling only.

Every function has the name and the argument order of its C entry point (include/shadowsync.h);
tensors are torch CUDA tensors, whose data pointers and the current torch stream are handed to C.
Nothing is computed here.  The library must have been built (``python -m paper_2003_03477_b200.build``
or ``__graft_entry__.build()``); a missing library is an error, there is no other execution path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libshadowsync.so")

SS_OK = 0
STATUS_NAMES = {0: "SS_OK", -1: "SS_ERR_NULL", -2: "SS_ERR_SHAPE", -3: "SS_ERR_ALIGN", -4: "SS_ERR_DTYPE",
                -5: "SS_ERR_WORKSPACE", -6: "SS_ERR_ARCH", -7: "SS_ERR_CUDA", -8: "SS_ERR_RANGE"}
SS_DEV_BAD_INDEX, SS_DEV_BAD_OFFSET, SS_DEV_BAD_WORKSPACE = 1, 2, 4
SS_TABLE_SORT_CAP = 24576          # lookups of one table that the light per-table sort takes (shadowsync.h)
SS_SYNC_EASGD_LITERAL = 1
SS_SYNC_BMUF_NESTEROV = 2

EXPORTS = ["ss_status_str", "ss_last_cuda_error", "ss_num_sms", "ss_embbag_fwd", "ss_embbag_bwd_workspace_bytes",
           "ss_embbag_bwd_adagrad", "ss_embbag_bwd_sort", "ss_embbag_bwd_apply", "ss_embbag_bwd_sort_noalloc", "ss_mlp_param_count", "ss_mlp_param_offsets", "ss_mlp_workspace_bytes",
           "ss_mlp_fwd", "ss_mlp_bwd", "ss_ne_accumulate", "ss_ne_value", "ss_sync_easgd", "ss_sync_ma", "ss_sync_bmuf", "ss_shadow_start", "ss_shadow_rounds", "ss_shadow_pause", "ss_shadow_stop", "ss_to_bf16",
           "ss_gemm_bf16", "ss_device_error", "ss_mlp_set_flow_ctas", "ssh_fill_uniform", "ss_profile", "ss_profile_collect"]


class SsError(RuntimeError):
    def __init__(self, fn: str, status: int, cuda_error: int = 0):
        self.status = status
        self.cuda_error = cuda_error
        msg = f"{fn}: {STATUS_NAMES.get(status, status)}"
        if status == -7:
            msg += f" (cudaError {cuda_error})"
        super().__init__(msg)


class MlpDesc(C.Structure):
    _fields_ = [("n_bottom", C.c_int), ("n_top", C.c_int), ("bottom_dims", C.POINTER(C.c_int)),
                ("top_dims", C.POINTER(C.c_int)), ("gemm_dtype", C.c_int)]


_lib = None


def lib() -> C.CDLL:
    """The loaded library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it first (python -m paper_2003_03477_b200.build); "
                               "there is no fallback path")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, f32, sz = C.c_void_p, C.c_int, C.c_int64, C.c_float, C.c_size_t
        L.ss_status_str.restype = C.c_char_p
        L.ss_status_str.argtypes = [i32]
        L.ss_last_cuda_error.restype = i32
        L.ss_num_sms.restype = i32
        L.ss_embbag_fwd.argtypes = [vp, i32, i64, i32, vp, vp, i32, vp, i64, vp, i64, i32, vp, vp]
        L.ss_embbag_bwd_workspace_bytes.restype = sz
        L.ss_embbag_bwd_workspace_bytes.argtypes = [i32, i64, i32, i32, i64]
        L.ss_embbag_bwd_adagrad.argtypes = [vp, vp, i32, i64, i32, vp, vp, i32, i64, vp, i64, i32, f32, f32,
                                            vp, sz, vp, vp, vp, vp, vp, vp]
        L.ss_embbag_bwd_sort.argtypes = [i32, i64, i32, vp, vp, i32, i64, vp, sz, vp, vp, vp, vp, vp, vp]
        L.ss_embbag_bwd_apply.argtypes = [vp, vp, i32, i64, i32, i32, i64, vp, i64, i32, f32, f32, vp, sz, vp, vp]
        L.ss_embbag_bwd_sort_noalloc.argtypes = [i32, i64, vp, vp, i32, i64, vp, vp, vp, vp, vp, vp]
        L.ss_mlp_param_count.restype = i64
        L.ss_mlp_param_count.argtypes = [C.POINTER(MlpDesc)]
        L.ss_mlp_param_offsets.argtypes = [C.POINTER(MlpDesc), C.POINTER(i64), C.POINTER(i64)]
        L.ss_mlp_workspace_bytes.restype = sz
        L.ss_mlp_workspace_bytes.argtypes = [C.POINTER(MlpDesc), i32]
        L.ss_mlp_fwd.argtypes = [C.POINTER(MlpDesc), vp, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp]
        L.ss_mlp_bwd.argtypes = [C.POINTER(MlpDesc), vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, f32, f32, i32,
                                 vp, i64, vp, sz, vp]
        L.ss_ne_accumulate.argtypes = [vp, vp, i32, vp, vp]
        L.ss_ne_value.argtypes = [vp, vp, vp]
        L.ss_sync_easgd.argtypes = [C.POINTER(vp), i32, vp, i64, f32, i32, C.POINTER(vp), vp]
        L.ss_sync_ma.argtypes = [C.POINTER(vp), i32, vp, i64, f32, i32, C.POINTER(vp), vp]
        L.ss_sync_bmuf.argtypes = [C.POINTER(vp), i32, vp, vp, i64, f32, f32, f32, i32, C.POINTER(vp), vp]
        L.ss_shadow_start.argtypes = [C.POINTER(vp), i32, C.POINTER(vp), i32, vp, vp, i64, f32, f32, f32, i32, C.POINTER(vp), vp,
                                      i32, i32, i64]
        L.ss_shadow_rounds.argtypes = [vp]
        L.ss_shadow_rounds.restype = i64
        L.ss_shadow_pause.argtypes = [vp, i32]
        L.ss_shadow_stop.argtypes = [vp, C.POINTER(i64)]
        L.ss_to_bf16.argtypes = [vp, vp, i64, vp]
        L.ss_gemm_bf16.argtypes = [vp, i32, i64, vp, i32, i64, vp, i64, i32, i32, i32, i32, vp]
        L.ss_device_error.argtypes = [i32]
        L.ss_mlp_set_flow_ctas.argtypes = [i32]
        L.ss_mlp_set_flow_ctas.restype = i32
        L.ss_profile.argtypes = [i32]
        L.ss_profile_collect.argtypes = [C.c_char_p, sz, C.POINTER(f32), i32]
        L.ssh_fill_uniform.argtypes = [vp, i64, C.c_uint64, C.c_uint64, f32, f32, vp]
        for name in EXPORTS:
            if name not in ("ss_status_str", "ss_last_cuda_error", "ss_num_sms", "ss_embbag_bwd_workspace_bytes",
                            "ss_mlp_param_count", "ss_mlp_workspace_bytes", "ss_shadow_rounds", "ss_mlp_set_flow_ctas"):
                getattr(L, name).restype = i32
        _lib = L
    return _lib


def _check(fn: str, status: int) -> None:
    if status != SS_OK:
        raise SsError(fn, status, lib().ss_last_cuda_error())


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    return t.data_ptr()


def _stream(stream) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream if hasattr(s, "cuda_stream") else int(s)


def _ptr_array(ts: Optional[Sequence[torch.Tensor]]):
    if ts is None:
        return None
    return (C.c_void_p * len(ts))(*[_ptr(t) for t in ts])


# ------------------------------------------------------------------------------------------
class MlpSpec:
    """Host description of the MLP (ss_mlp_desc) with the flat parameter layout the library reports."""

    def __init__(self, bottom_dims: Sequence[int], top_dims: Sequence[int], bf16: bool):
        self.bottom_dims, self.top_dims, self.bf16 = tuple(bottom_dims), tuple(top_dims), bool(bf16)
        self._b = (C.c_int * len(self.bottom_dims))(*self.bottom_dims)
        self._t = (C.c_int * len(self.top_dims))(*self.top_dims)
        self.desc = MlpDesc(len(self.bottom_dims) - 1, len(self.top_dims) - 1, self._b, self._t, 1 if bf16 else 0)
        self.n_layers = self.desc.n_bottom + self.desc.n_top
        self.param_count = ss_mlp_param_count(self)
        if self.param_count < 0:
            raise SsError("ss_mlp_param_count", -2)
        w = (C.c_int64 * self.n_layers)()
        b = (C.c_int64 * self.n_layers)()
        _check("ss_mlp_param_offsets", lib().ss_mlp_param_offsets(C.byref(self.desc), w, b))
        self.w_off, self.b_off = list(w), list(b)
        dims = []
        for d in (self.bottom_dims, self.top_dims):
            dims += [(d[i], d[i + 1]) for i in range(len(d) - 1)]
        self.layer_dims = dims          # (in, out) per layer

    @property
    def D0(self) -> int:
        return self.bottom_dims[-1]

    @property
    def W(self) -> int:
        return self.top_dims[0]


def ss_status_str(status: int) -> str:
    return lib().ss_status_str(status).decode()


def ss_num_sms() -> int:
    return lib().ss_num_sms()


def ss_mlp_param_count(spec: MlpSpec) -> int:
    return lib().ss_mlp_param_count(C.byref(spec.desc))


def ss_mlp_workspace_bytes(spec: MlpSpec, B: int) -> int:
    return lib().ss_mlp_workspace_bytes(C.byref(spec.desc), B)


def ss_embbag_bwd_workspace_bytes(T: int, N: int, D: int, B: int, L: int) -> int:
    return lib().ss_embbag_bwd_workspace_bytes(T, N, D, B, L)


def ss_embbag_fwd(tables, T, N, D, indices, offsets, B, out_f32, ld_f32, out_bf16, ld_bf16, col0, d_status,
                  stream=None) -> None:
    _check("ss_embbag_fwd", lib().ss_embbag_fwd(_ptr(tables), T, N, D, _ptr(indices), _ptr(offsets), B,
                                                 _ptr(out_f32), ld_f32, _ptr(out_bf16), ld_bf16, col0,
                                                 _ptr(d_status), _stream(stream)))


def ss_embbag_bwd_adagrad(tables, row_state, T, N, D, indices, offsets, B, L, grad, ld_grad, col0, lr, eps,
                          workspace, uniq_keys, seg_off, perm, d_num_unique, d_status, stream=None) -> None:
    _check("ss_embbag_bwd_adagrad",
           lib().ss_embbag_bwd_adagrad(_ptr(tables), _ptr(row_state), T, N, D, _ptr(indices), _ptr(offsets), B, L,
                                       _ptr(grad), ld_grad, col0, lr, eps, _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _ptr(uniq_keys), _ptr(seg_off),
                                       _ptr(perm), _ptr(d_num_unique), _ptr(d_status), _stream(stream)))


def ss_embbag_bwd_sort(T, N, D, indices, offsets, B, L, workspace, uniq_keys, seg_off, perm, d_num_unique, d_status,
                       stream=None) -> None:
    _check("ss_embbag_bwd_sort",
           lib().ss_embbag_bwd_sort(T, N, D, _ptr(indices), _ptr(offsets), B, L, _ptr(workspace),
                                    workspace.numel() * workspace.element_size(), _ptr(uniq_keys), _ptr(seg_off),
                                    _ptr(perm), _ptr(d_num_unique), _ptr(d_status), _stream(stream)))


def ss_embbag_bwd_apply(tables, row_state, T, N, D, B, L, grad, ld_grad, col0, lr, eps, workspace, d_status=None,
                        stream=None) -> None:
    _check("ss_embbag_bwd_apply",
           lib().ss_embbag_bwd_apply(_ptr(tables), _ptr(row_state), T, N, D, B, L, _ptr(grad), ld_grad, col0, lr, eps,
                                     _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(d_status),
                                     _stream(stream)))


def ss_embbag_bwd_sort_noalloc(T, N, indices, offsets, B, L, uniq_keys, seg_off, perm, d_num_unique, d_status,
                               stream=None) -> None:
    """Sort / unique with the library's built-in scratch (no workspace, nothing allocated); L <= 65536."""
    _check("ss_embbag_bwd_sort_noalloc",
           lib().ss_embbag_bwd_sort_noalloc(T, N, _ptr(indices), _ptr(offsets), B, L, _ptr(uniq_keys), _ptr(seg_off),
                                            _ptr(perm), _ptr(d_num_unique), _ptr(d_status), _stream(stream)))


def ss_mlp_fwd(spec: MlpSpec, w, w_bf16, dense, concat_f32, concat_bf16, B, labels, logit, prob, loss, workspace,
               stream=None) -> None:
    _check("ss_mlp_fwd", lib().ss_mlp_fwd(C.byref(spec.desc), _ptr(w), _ptr(w_bf16), _ptr(dense), _ptr(concat_f32),
                                           _ptr(concat_bf16), B, _ptr(labels), _ptr(logit), _ptr(prob), _ptr(loss),
                                           _ptr(workspace), workspace.numel() * workspace.element_size(),
                                           _stream(stream)))


def ss_mlp_bwd(spec: MlpSpec, w, w_bf16, adagrad_acc, grads, dense, concat_f32, concat_bf16, labels, prob, B, lr,
               eps, apply_update, grad_pooled, ld_grad, workspace, stream=None) -> None:
    _check("ss_mlp_bwd", lib().ss_mlp_bwd(C.byref(spec.desc), _ptr(w), _ptr(w_bf16), _ptr(adagrad_acc), _ptr(grads),
                                           _ptr(dense), _ptr(concat_f32), _ptr(concat_bf16), _ptr(labels), _ptr(prob),
                                           B, lr, eps, int(apply_update), _ptr(grad_pooled), ld_grad, _ptr(workspace),
                                           workspace.numel() * workspace.element_size(), _stream(stream)))


def ss_ne_accumulate(logit, labels, B, acc, stream=None) -> None:
    _check("ss_ne_accumulate", lib().ss_ne_accumulate(_ptr(logit), _ptr(labels), B, _ptr(acc), _stream(stream)))


def ss_ne_value(acc, out, stream=None) -> None:
    _check("ss_ne_value", lib().ss_ne_value(_ptr(acc), _ptr(out), _stream(stream)))


def ss_sync_easgd(w: Sequence[torch.Tensor], center, n, alpha, flags=0, w_bf16=None, stream=None) -> None:
    _check("ss_sync_easgd", lib().ss_sync_easgd(_ptr_array(w), len(w), _ptr(center), n, alpha, flags,
                                                 _ptr_array(w_bf16), _stream(stream)))


def ss_sync_ma(w: Sequence[torch.Tensor], global_out, n, alpha, flags=0, w_bf16=None, stream=None) -> None:
    _check("ss_sync_ma", lib().ss_sync_ma(_ptr_array(w), len(w), _ptr(global_out), n, alpha, flags,
                                           _ptr_array(w_bf16), _stream(stream)))


def ss_sync_bmuf(w: Sequence[torch.Tensor], global_, delta, n, alpha, eta, mu, flags=0, w_bf16=None,
                 stream=None) -> None:
    _check("ss_sync_bmuf", lib().ss_sync_bmuf(_ptr_array(w), len(w), _ptr(global_), _ptr(delta), n, alpha, eta, mu,
                                               flags, _ptr_array(w_bf16), _stream(stream)))


def ss_gemm_bf16(a, a_mn_major, lda, b, b_mn_major, ldb, c, ldc, M, N, K, force_simt=0, stream=None) -> None:
    _check("ss_gemm_bf16", lib().ss_gemm_bf16(_ptr(a), int(a_mn_major), lda, _ptr(b), int(b_mn_major), ldb, _ptr(c),
                                               ldc, M, N, K, int(force_simt), _stream(stream)))


def ss_mlp_set_flow_ctas(ctas: int) -> int:
    """CTAs the persistent tensor-core launches of the MLP take (0 = the library's default, negative = leave as it
    is); returns the number now in effect."""
    return int(lib().ss_mlp_set_flow_ctas(int(ctas)))


def ss_device_error(clear: bool = True) -> int:
    return lib().ss_device_error(1 if clear else 0)


RULES = {"easgd": 0, "ma": 1, "bmuf": 2}


def ss_shadow_start(rule, w, center, delta, n, alpha, eta=1.0, mu=0.0, flags=0, w_bf16=None, stream=None,
                    max_in_flight=2, pause_us=0, max_rounds=1 << 40):
    """Start the native shadow thread; returns its handle (pass it to ss_shadow_rounds / ss_shadow_stop)."""
    h = C.c_void_p()
    _check("ss_shadow_start", lib().ss_shadow_start(C.byref(h), RULES[rule], _ptr_array(w), len(w), _ptr(center),
                                                     _ptr(delta), n, alpha, eta, mu, flags, _ptr_array(w_bf16),
                                                     _stream(stream), max_in_flight, pause_us, max_rounds))
    return h


def ss_shadow_rounds(handle) -> int:
    return int(lib().ss_shadow_rounds(handle))


def ss_shadow_pause(handle, paused: bool) -> None:
    """paused=True: stop enqueuing and return once every enqueued pass has completed; False: loop again."""
    _check("ss_shadow_pause", lib().ss_shadow_pause(handle, 1 if paused else 0))


def ss_shadow_stop(handle) -> int:
    """Stop and join the shadow thread; returns the number of synchronisation passes it enqueued."""
    rounds = C.c_int64(0)
    _check("ss_shadow_stop", lib().ss_shadow_stop(handle, C.byref(rounds)))
    return int(rounds.value)


def ss_to_bf16(src, dst_bf16, n, stream=None) -> None:
    _check("ss_to_bf16", lib().ss_to_bf16(_ptr(src), _ptr(dst_bf16), n, _stream(stream)))


def ssh_fill_uniform(dst, count, key, counter0, scale, mid, stream=None) -> None:
    _check("ssh_fill_uniform", lib().ssh_fill_uniform(_ptr(dst), count, int(key), int(counter0), scale, mid,
                                                       _stream(stream)))


def ss_profile(on: bool) -> bool:
    """Switch the library's per-kernel timers on or off (off while capturing CUDA graphs)."""
    return bool(lib().ss_profile(1 if on else 0))


def ss_profile_collect(max_records: int = 1 << 16):
    """[(kernel name, milliseconds)] of every launch timed since the last collect, in launch order."""
    names = C.create_string_buffer(max_records * 32)
    ms = (C.c_float * max_records)()
    n = lib().ss_profile_collect(names, len(names), ms, max_records)
    if n < 0:
        raise SsError("ss_profile_collect", -7, lib().ss_last_cuda_error())
    return list(zip(names.value.decode().split("\n")[:n], list(ms[:n])))
