"""ctypes binding of the C ABI in include/prhs.h.

Argument marshalling only: every step of the path runs in the CUDA library.  Tensors are
passed as raw device (or host) pointers; torch is used for device memory and streams.
Loading fails loudly if the library has not been built -- there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libprhs.so")

PRHS_OK = 0
STATUS_NAMES = {0: "PRHS_OK", 1: "PRHS_ERR_INVALID_ARG", 2: "PRHS_ERR_UNSUPPORTED", 3: "PRHS_ERR_OOM",
                4: "PRHS_ERR_CUDA", 5: "PRHS_ERR_STATE", 6: "PRHS_ERR_CAPACITY",
                7: "PRHS_ERR_DEVICE_FLAG"}
PRHS_DILATE_ANCHOR = 1
PRHS_WANT_DELTA = 2
PRHS_GROUP_SETS = 4
PRHS_FLAG_BAD_INDEX, PRHS_FLAG_BAD_PAGE, PRHS_FLAG_SELECT_FALLBACK, PRHS_FLAG_TIMEOUT = 1, 2, 4, 8
PRHS_CFG_NO_TMA = 1
PRHS_CFG_TMA_GATHER = 2
PRHS_CFG_MMA_SYNC_SCORE = 4
PRHS_CFG_GROUP_TCGEN05 = 8

# every symbol include/prhs.h declares
EXPORTS = ["prhs_create", "prhs_destroy", "prhs_score_topk", "prhs_build_index_set",
           "prhs_sparse_decode_attn", "prhs_dense_decode_attn", "prhs_decode_step",
           "prhs_decode_step_host", "prhs_decode_step_host_async", "prhs_delta", "prhs_index_capacity", "prhs_get_index_set",
           "prhs_get_shared_set", "prhs_get_scores", "prhs_scores_ld", "prhs_check",
           "prhs_launch_count", "prhs_selftest_wait", "prhs_state_bytes", "prhs_state_export", "prhs_state_import", "prhs_validate_index_lists", "prhs_last_error", "prhs_version", "prhs_profile_begin",
           "prhs_profile_end", "prhs_kernel_kind_name", "prhs_sparse_decode_attn_noalloc", "prhs_get_gate",
           "prhs_noalloc_check", "prhs_gather_probe"]
NOALLOC_MAX_UNITS = 1024
KERNEL_KINDS = 6


class PrhsError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "num_layers", "max_batch", "num_q_heads", "num_kv_heads", "head_dim", "max_context",
        "page_size", "max_k", "max_window", "max_sinks", "max_dilate_r", "max_dilate_m",
        "min_layer_group", "max_block_sets")] + [("flags", C.c_uint32)]


class KvView(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("stride_outer", C.c_int64),
                ("stride_head", C.c_int64), ("page_table", C.c_void_p),
                ("page_table_stride", C.c_int32), ("seq_lens", C.c_void_p),
                ("max_seq_len", C.c_int32), ("num_pages", C.c_int32)]


class Schedule(C.Structure):
    _fields_ = [("refresh_interval", C.c_int32), ("layer_group", C.c_int32), ("top_k", C.c_int32),
                ("top_k_per_seq", C.c_void_p), ("window", C.c_int32), ("sinks", C.c_int32),
                ("dilate_r", C.c_int32), ("dilate_m", C.c_int32), ("flags", C.c_uint32),
                ("psaw_phi", C.c_float), ("psaw_alpha", C.c_float), ("psaw_layer_start", C.c_int32),
                ("sim_threshold", C.c_float)]


_lib = None


def load() -> C.CDLL:
    """Load libprhs.so (built by `paper_2602_08329_b200.build`); raise if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2602_08329_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, st = C.c_void_p, C.c_int32, C.c_int
    sig = {
        "prhs_create": (st, [C.POINTER(Config), C.POINTER(vp)]),
        "prhs_destroy": (st, [vp]),
        "prhs_score_topk": (st, [vp, i32, i32, vp, C.POINTER(KvView), C.POINTER(Schedule), i32, vp, vp, vp, vp]),
        "prhs_build_index_set": (st, [vp, i32, i32, C.POINTER(Schedule), C.POINTER(KvView), i32, vp, i32, vp, vp]),
        "prhs_sparse_decode_attn": (st, [vp, vp, C.POINTER(KvView), vp, vp, i32, i32, vp, vp, vp]),
        "prhs_dense_decode_attn": (st, [vp, vp, C.POINTER(KvView), i32, vp, vp, vp]),
        "prhs_sparse_decode_attn_noalloc": (st, [vp, C.POINTER(KvView), vp, vp, i32, i32, i32, i32, vp, vp, vp]),
        "prhs_noalloc_check": (st, [vp, C.POINTER(C.c_uint32)]),
        "prhs_gather_probe": (st, [vp, i32, C.POINTER(KvView), vp, vp, i32, i32, vp]),
        "prhs_decode_step": (st, [vp, i32, i32, C.POINTER(Schedule), vp, C.POINTER(KvView), i32, vp, vp, vp]),
        "prhs_decode_step_host": (st, [vp, i32, i32, C.POINTER(Schedule), vp, vp, vp, vp, C.POINTER(KvView), i32, vp, vp]),
        "prhs_decode_step_host_async": (st, [vp, i32, i32, C.POINTER(Schedule), vp, vp, vp, vp, C.POINTER(KvView), i32,
                                              vp, vp]),
        "prhs_delta": (st, [vp, vp, C.POINTER(KvView), vp, vp, i32, i32, vp, vp]),
        "prhs_index_capacity": (i32, [vp]),
        "prhs_get_index_set": (st, [vp, i32, vp, vp, vp]),
        "prhs_get_shared_set": (st, [vp, i32, i32, vp, vp, vp, vp, vp]),
        "prhs_get_scores": (st, [vp, i32, vp, vp]),
        "prhs_get_gate": (st, [vp, i32, i32, vp, vp, vp]),
        "prhs_scores_ld": (i32, [vp]),
        "prhs_check": (st, [vp, vp, C.POINTER(C.c_uint32)]),
        "prhs_profile_begin": (st, [vp, i32]),
        "prhs_profile_end": (st, [vp, vp, C.POINTER(C.c_float), C.POINTER(C.c_int64)]),
        "prhs_kernel_kind_name": (C.c_char_p, [i32]),
        "prhs_launch_count": (C.c_int64, [vp]),
        "prhs_validate_index_lists": (st, [vp, C.POINTER(KvView), vp, vp, i32, i32, vp, C.POINTER(C.c_int32), vp]),
        "prhs_state_bytes": (C.c_int64, [vp]),
        "prhs_state_export": (st, [vp, vp, C.c_int64, vp]),
        "prhs_state_import": (st, [vp, vp, C.c_int64, vp]),
        "prhs_selftest_wait": (st, [vp, C.c_int64, C.POINTER(C.c_int32), vp]),
        "prhs_last_error": (C.c_char_p, [vp]),
        "prhs_version": (C.c_char_p, []),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous(), "tensors passed to the library must be contiguous"
        return t.data_ptr()
    return int(t)


def _stream(stream=None):
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def make_schedule(top_k, window, sinks, refresh_interval=1, layer_group=1, dilate_r=1, dilate_m=-1,
                  top_k_per_seq=None, flags=0, psaw_phi=0.7, psaw_alpha=1.0, psaw_layer_start=0,
                  sim_threshold=-1.0) -> Schedule:
    s = Schedule(refresh_interval, layer_group, top_k, _ptr(top_k_per_seq), window, sinks,
                 dilate_r, dilate_m, flags, psaw_phi, psaw_alpha, psaw_layer_start, sim_threshold)
    s._keep = top_k_per_seq
    return s


def make_view(k, v, seq_lens, page_table=None, max_seq_len=0) -> KvView:
    """View of a cache tensor: contiguous [B][Hkv][cap][128] or paged [pool][Hkv][16][128]."""
    assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and k.shape[-1] == 128
    assert k.stride() == v.stride() and k.stride(-1) == 1 and k.stride(-2) == 128
    assert seq_lens.dtype == torch.int32
    view = KvView(k.data_ptr(), v.data_ptr(), k.stride(0), k.stride(1),
                  _ptr(page_table), page_table.stride(0) if page_table is not None else 0,
                  seq_lens.data_ptr(), max_seq_len, k.shape[0] if page_table is not None else 0)
    view._keep = (k, v, seq_lens, page_table)
    return view


class Context:
    """Owns a prhs_ctx.  Methods mirror the C entry points one to one."""

    def __init__(self, num_layers, max_batch, num_q_heads, num_kv_heads, max_context, max_k,
                 max_window, max_sinks, max_dilate_r=1, max_dilate_m=-1, page_size=0,
                 min_layer_group=1, head_dim=128, max_block_sets=1, flags=0):
        self.lib = load()
        self.cfg = Config(num_layers, max_batch, num_q_heads, num_kv_heads, head_dim, max_context,
                          page_size, max_k, max_window, max_sinks, max_dilate_r, max_dilate_m,
                          min_layer_group, max_block_sets, flags)
        h = C.c_void_p()
        rc = self.lib.prhs_create(C.byref(self.cfg), C.byref(h))
        if rc != PRHS_OK:
            raise PrhsError(rc, self.lib.prhs_last_error(None).decode())
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            self.lib.prhs_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _ck(self, rc):
        if rc != PRHS_OK:
            raise PrhsError(rc, self.lib.prhs_last_error(self.h).decode())

    # -- sizes
    @property
    def index_capacity(self) -> int:
        return self.lib.prhs_index_capacity(self.h)

    @property
    def scores_ld(self) -> int:
        return self.lib.prhs_scores_ld(self.h)

    @property
    def launch_count(self) -> int:
        return self.lib.prhs_launch_count(self.h)

    # -- entry points
    def score_topk(self, layer, step, q, view, sched, batch, out_idx=None, out_count=None,
                   out_lse_full=None, stream=None):
        self._ck(self.lib.prhs_score_topk(self.h, layer, step, _ptr(q), C.byref(view), C.byref(sched),
                                          batch, _ptr(out_idx), _ptr(out_count), _ptr(out_lse_full),
                                          _stream(stream)))

    def build_index_set(self, layer, step, sched, view, batch, out_idx, out_count, stream=None):
        self._ck(self.lib.prhs_build_index_set(self.h, layer, step, C.byref(sched), C.byref(view), batch,
                                               _ptr(out_idx), out_idx.shape[-1], _ptr(out_count),
                                               _stream(stream)))

    def sparse_decode_attn(self, q, view, idx, count, batch, out, out_lse=None, stream=None):
        self._ck(self.lib.prhs_sparse_decode_attn(self.h, _ptr(q), C.byref(view), _ptr(idx), _ptr(count),
                                                  idx.shape[-1], batch, _ptr(out), _ptr(out_lse),
                                                  _stream(stream)))

    def gather_probe(self, variant, view, idx, count, batch, stream=None):
        """The bare row gather of sparse_decode_attn (measurement support; see prhs_gather_probe)."""
        self._ck(self.lib.prhs_gather_probe(self.h, variant, C.byref(view), _ptr(idx), _ptr(count), idx.shape[-1],
                                            batch, _stream(stream)))

    def dense_decode_attn(self, q, view, batch, out, out_lse=None, stream=None):
        self._ck(self.lib.prhs_dense_decode_attn(self.h, _ptr(q), C.byref(view), batch, _ptr(out),
                                                 _ptr(out_lse), _stream(stream)))

    def decode_step(self, layer, step, sched, q, view, batch, out, out_delta=None, stream=None):
        self._ck(self.lib.prhs_decode_step(self.h, layer, step, C.byref(sched), _ptr(q), C.byref(view),
                                           batch, _ptr(out), _ptr(out_delta), _stream(stream)))

    def decode_step_host(self, layer, step, sched, host_q, host_new_k, host_new_v, host_seq_lens,
                         view, batch, host_out, stream=None, sync=True):
        fn = self.lib.prhs_decode_step_host if sync else self.lib.prhs_decode_step_host_async
        self._ck(fn(self.h, layer, step, C.byref(sched), _ptr(host_q), _ptr(host_new_k), _ptr(host_new_v),
                    _ptr(host_seq_lens), C.byref(view), batch, _ptr(host_out), _stream(stream)))

    def delta(self, q, view, idx, count, batch, out_delta, stream=None):
        self._ck(self.lib.prhs_delta(self.h, _ptr(q), C.byref(view), _ptr(idx), _ptr(count),
                                     idx.shape[-1], batch, _ptr(out_delta), _stream(stream)))

    def get_index_set(self, batch, stream=None):
        hq, cap = self.cfg.num_q_heads, self.index_capacity
        idx = torch.empty(batch, hq, cap, dtype=torch.int32)
        cnt = torch.empty(batch, hq, dtype=torch.int32)
        self._ck(self.lib.prhs_get_index_set(self.h, batch, idx.data_ptr(), cnt.data_ptr(), _stream(stream)))
        return idx, cnt

    def get_shared_set(self, layer, batch, stream=None):
        hq, mk = self.cfg.num_q_heads, self.cfg.max_k
        hat_cap = self.index_capacity - self.cfg.max_sinks - self.cfg.max_window
        s_star = torch.empty(batch, hq, mk, dtype=torch.int32)
        n_star = torch.empty(batch, hq, dtype=torch.int32)
        s_hat = torch.empty(batch, hq, hat_cap, dtype=torch.int32)
        n_hat = torch.empty(batch, hq, dtype=torch.int32)
        self._ck(self.lib.prhs_get_shared_set(self.h, layer, batch, s_star.data_ptr(), n_star.data_ptr(),
                                              s_hat.data_ptr(), n_hat.data_ptr(), _stream(stream)))
        return s_star, n_star, s_hat, n_hat

    def get_gate(self, layer, batch, stream=None):
        need = torch.empty(batch, self.cfg.num_q_heads, dtype=torch.int32)
        ref = torch.empty(batch, self.cfg.num_q_heads, dtype=torch.int32)
        self._ck(self.lib.prhs_get_gate(self.h, layer, batch, need.data_ptr(), ref.data_ptr(), _stream(stream)))
        return need, ref

    def get_scores(self, batch, stream=None):
        out = torch.empty(batch, self.cfg.num_q_heads, self.scores_ld, dtype=torch.float32)
        self._ck(self.lib.prhs_get_scores(self.h, batch, out.data_ptr(), _stream(stream)))
        return out

    def profile_begin(self, max_launches=4096):
        self._ck(self.lib.prhs_profile_begin(self.h, max_launches))

    def profile_end(self, stream=None) -> dict:
        """{kind name: (total ms, launches)} for the launches since profile_begin."""
        ms = (C.c_float * KERNEL_KINDS)()
        n = (C.c_int64 * KERNEL_KINDS)()
        self._ck(self.lib.prhs_profile_end(self.h, _stream(stream), ms, n))
        return {self.lib.prhs_kernel_kind_name(i).decode(): (float(ms[i]), int(n[i]))
                for i in range(KERNEL_KINDS)}

    def validate_index_lists(self, view, idx, count, batch, stream=None):
        """(number of bad units, CPU int32 [batch][Hq] marks) for explicit index lists."""
        marks = torch.empty(batch, self.cfg.num_q_heads, dtype=torch.int32)
        nbad = C.c_int32(-1)
        self._ck(self.lib.prhs_validate_index_lists(self.h, C.byref(view), _ptr(idx), _ptr(count), idx.shape[-1],
                                                    batch, marks.data_ptr(), C.byref(nbad), _stream(stream)))
        return nbad.value, marks

    def state_export(self, stream=None) -> torch.Tensor:
        """The shared-set state as a flat CPU uint8 tensor (see prhs_state_export)."""
        buf = torch.empty(self.lib.prhs_state_bytes(self.h), dtype=torch.uint8)
        self._ck(self.lib.prhs_state_export(self.h, buf.data_ptr(), buf.numel(), _stream(stream)))
        return buf

    def state_import(self, buf: torch.Tensor, stream=None):
        assert buf.dtype == torch.uint8 and buf.device.type == "cpu" and buf.is_contiguous()
        self._ck(self.lib.prhs_state_import(self.h, buf.data_ptr(), buf.numel(), _stream(stream)))

    def selftest_wait(self, budget_cycles=1_000_000, stream=None) -> int:
        gave_up = C.c_int32(-1)
        self._ck(self.lib.prhs_selftest_wait(self.h, budget_cycles, C.byref(gave_up), _stream(stream)))
        return gave_up.value

    def check(self, stream=None) -> int:
        flags = C.c_uint32(0)
        self._ck(self.lib.prhs_check(self.h, _stream(stream), C.byref(flags)))
        return flags.value


def sparse_decode_attn_noalloc(q, view, idx, count, batch, num_q_heads, num_kv_heads, out, out_lse=None,
                               stream=None):
    """The context-free, allocation-free variant of Context.sparse_decode_attn.

    For callers that may not allocate device memory (a frozen memory budget, a framework
    that owns the heap): it needs no Context, and its scratch is a fixed array inside the
    library.  Raises PrhsError on a shape beyond the array's capacity.
    """
    lib = load()
    rc = lib.prhs_sparse_decode_attn_noalloc(_ptr(q), C.byref(view), _ptr(idx), _ptr(count), idx.shape[-1],
                                             batch, num_q_heads, num_kv_heads, _ptr(out), _ptr(out_lse),
                                             _stream(stream))
    if rc != PRHS_OK:
        raise PrhsError(rc, lib.prhs_last_error(None).decode())


def noalloc_check(stream=None) -> int:
    """Report and clear the anomaly word of the allocation-free calls on the current device.

    Returns 0 when clean; raises PrhsError (PRHS_ERR_DEVICE_FLAG) when a call skipped an index
    outside [0, t_b) or a page id outside the pool.  Synchronises the stream.
    """
    lib = load()
    flags = C.c_uint32(0)
    rc = lib.prhs_noalloc_check(_stream(stream), C.byref(flags))
    if rc != PRHS_OK:
        raise PrhsError(rc, lib.prhs_last_error(None).decode())
    return flags.value


def version() -> str:
    return load().prhs_version().decode()
