"""ctypes binding of libqevict.so: the same entry points as include/qevict.h, plus a small convenience
class that owns the device workspace.  Argument marshalling only -- every step of the path runs in the
CUDA kernels of the library; there is no fallback of any kind."""

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqevict.so")
# QEVICT_TRACE_LIB=1 loads the tracing variant (build.build(trace=True)): the same kernels plus %globaltimer
# stamps, which qevict_kernel_timeline reads.  It is a measuring aid; numbers reported as throughput come from
# the normal library.
if os.environ.get("QEVICT_TRACE_LIB", "0") not in ("", "0"):
    LIB_PATH = os.path.join(_HERE, "libqevict_trace.so")
# QEVICT_CHECK_LIB=1 loads the checking variant (build.build(variant="check")): the same kernels with every table
# index range-checked before use and the pools poisoned with NaN at creation.
if os.environ.get("QEVICT_CHECK_LIB", "0") not in ("", "0"):
    LIB_PATH = os.path.join(_HERE, "libqevict_check.so")

QEVICT_OK = 0
DTYPE_FP16, DTYPE_BF16 = 0, 1
(QEVICT_TIER_NONE, QEVICT_TIER_OPEN, QEVICT_TIER_AGED, QEVICT_TIER_FULL, QEVICT_TIER_QUANT, QEVICT_TIER_EVICTED,
 QEVICT_TIER_SINK) = range(7)
QEVICT_RANK_CUMULATIVE, QEVICT_RANK_DECAYED, QEVICT_RANK_PNORM, QEVICT_RANK_KEYNORM = range(4)
TIER_NONE, TIER_OPEN, TIER_AGED, TIER_FULL, TIER_QUANT, TIER_EVICTED = range(6)
LEDGER_NONE, LEDGER_ACTIVE, LEDGER_DORMANT = range(3)
STATUS_NAMES = ["OK", "INVALID_ARG", "BAD_STATE", "NO_MEMORY", "UNSUPPORTED", "CUDA", "DEVICE_CHECK"]


class QEvictError(RuntimeError):
    def __init__(self, status, message):
        super().__init__("qevict: %s (%s)" % (message, STATUS_NAMES[status] if 0 <= status < 7 else status))
        self.status = status


class qevict_config(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("batch", C.c_int32), ("n_layers", C.c_int32), ("n_q_heads", C.c_int32),
        ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("dtype", C.c_int32), ("window", C.c_int32),
        ("quant_bits", C.c_int32), ("group_size", C.c_int32), ("fp_budget_windows", C.c_int32),
        ("q_budget_windows", C.c_int32), ("max_context", C.c_int32), ("rebalance_interval_hint", C.c_int32),
        ("softmax_scale", C.c_float), ("device", C.c_int32), ("sink_windows", C.c_int32), ("recent_windows", C.c_int32),
        ("rank_mode", C.c_int32), ("rank_param", C.c_float), ("one_way", C.c_int32), ("rope_base", C.c_float),
    ]


class qevict_stats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in (
        "promotions", "quantizations", "reactivations", "deletions", "n_full", "n_quant", "n_aged", "n_open",
        "n_evicted", "decode_steps", "n_sink")]


class qevict_state_layout(C.Structure):
    _fields_ = [("n_window_slots", C.c_int32), ("n_fp_pages", C.c_int32), ("n_q_pages", C.c_int32), ("n_entries", C.c_int32),
                ("fp_pool_bytes", C.c_uint64), ("q_pool_bytes", C.c_uint64)]


_STATE_SCALARS = ("n_windows", "open_window", "open_fill", "n_live", "layer_prefilled", "layer_has_open", "layer_open_fill",
                  "layer_n_windows", "layer_aged")
_STATE_ARRAYS = ("tier", "ledger", "fp_page", "q_page", "importance", "event_mass", "fp_owner", "q_owner", "entries",
                 "last_mass", "fp_pool", "q_pool")


class qevict_state_view(C.Structure):
    _fields_ = ([("struct_size", C.c_uint32)] + [(n, C.c_int32) for n in _STATE_SCALARS] +
                [("knorm_acc", C.c_float), ("counters", C.c_uint64 * 4), ("decode_steps", C.c_uint64)] +
                [(n, C.c_void_p) for n in _STATE_ARRAYS])


_lib = None

_SIGNATURES = {
    "qevict_version": (C.c_char_p, []),
    "qevict_build_flavour": (C.c_int32, []),
    "qevict_status_string": (C.c_char_p, [C.c_int]),
    "qevict_last_error": (C.c_char_p, [C.c_void_p]),
    "qevict_launch_count": (C.c_uint64, [C.c_void_p]),
    "qevict_budget_from_bytes": (C.c_int, [C.POINTER(qevict_config), C.c_uint64, C.c_double, C.POINTER(C.c_int32),
                                           C.POINTER(C.c_int32), C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]),
    "qevict_workspace_bytes": (C.c_int, [C.POINTER(qevict_config), C.POINTER(C.c_uint64)]),
    "qevict_create": (C.c_int, [C.POINTER(qevict_config), C.c_void_p, C.c_uint64, C.POINTER(C.c_void_p)]),
    "qevict_destroy": (C.c_int, [C.c_void_p]),
    "qevict_set_splits": (C.c_int, [C.c_void_p, C.c_int32]),
    "qevict_prefill_score_scratch_bytes": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.POINTER(C.c_uint64)]),
    "qevict_prefill_score": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                      C.c_uint64, C.c_void_p]),
    "qevict_export_event_mass": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]),
    "qevict_set_kernel_timing": (C.c_int, [C.c_void_p, C.c_int32]),
    "qevict_kernel_time": (C.c_int, [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_uint64)]),
    "qevict_kernel_times": (C.c_int, [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_uint64)]),
    "qevict_kernel_timeline": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_double),
                                        C.POINTER(C.c_double), C.POINTER(C.c_int32)]),
    "qevict_prefill_assign": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "qevict_decode_attn": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "qevict_decode_attn_host": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "qevict_decode_attn_host_async": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "qevict_decode_attn_noalloc": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "qevict_wait_result": (C.c_int, [C.c_void_p]),
    "qevict_rebalance": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p]),
    "qevict_state_layout_of": (C.c_int, [C.c_void_p, C.POINTER(qevict_state_layout)]),
    "qevict_export_state": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.POINTER(qevict_state_view)]),
    "qevict_import_state": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.POINTER(qevict_state_view)]),
    "qevict_get_stats": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(qevict_stats)]),
    "qevict_check_device": (C.c_int, [C.c_void_p, C.POINTER(C.c_int32)]),
    "qevict_export_tables": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32] + [C.c_void_p] * 7),
    "qevict_export_last_mass": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]),
    "qevict_export_fp_page": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]),
    "qevict_export_q_page": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32] + [C.c_void_p] * 5),
}


def lib():
    """The loaded shared library.  Raises if it has not been built (there is no other code path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(os.path.basename(LIB_PATH) + " is missing: run `python -m paper_2608_05326_b200.build` "
                               "(or __graft_entry__.build()) first; there is no fallback path")
        handle = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


def _check(status, handle=None):
    if status != QEVICT_OK:
        # without a handle: the calling thread's last failure of qevict_create / qevict_workspace_bytes
        msg = lib().qevict_last_error(handle).decode()
        raise QEvictError(status, msg or lib().qevict_status_string(status).decode())


def make_config(batch, n_layers, n_q_heads, n_kv_heads, head_dim, dtype, window, quant_bits, group_size,
                fp_budget_windows, q_budget_windows, max_context, rebalance_interval_hint=0, softmax_scale=0.0,
                device=0, sink_windows=0, recent_windows=0, rank_mode=0, rank_param=0.0, one_way=0, rope_base=0.0):
    dt = {"fp16": DTYPE_FP16, "bf16": DTYPE_BF16, torch.float16: DTYPE_FP16, torch.bfloat16: DTYPE_BF16}[dtype]
    return qevict_config(C.sizeof(qevict_config), batch, n_layers, n_q_heads, n_kv_heads, head_dim, dt, window,
                         quant_bits, group_size, fp_budget_windows, q_budget_windows, max_context,
                         rebalance_interval_hint, softmax_scale, device, sink_windows, recent_windows, rank_mode,
                         rank_param, int(one_way), float(rope_base))


# --- plain function wrappers, same names as the C entry points -----------------------------------------
def qevict_version():
    return lib().qevict_version().decode()


def qevict_budget_from_bytes(cfg, hist_bytes, q_frac):
    kf, kq, mf, mq = C.c_int32(), C.c_int32(), C.c_uint64(), C.c_uint64()
    _check(lib().qevict_budget_from_bytes(C.byref(cfg), int(hist_bytes), float(q_frac), C.byref(kf), C.byref(kq),
                                          C.byref(mf), C.byref(mq)))
    return kf.value, kq.value, mf.value, mq.value


def qevict_workspace_bytes(cfg):
    n = C.c_uint64()
    _check(lib().qevict_workspace_bytes(C.byref(cfg), C.byref(n)))
    return n.value


def qevict_create(cfg, device_mem_ptr, n_bytes):
    h = C.c_void_p()
    _check(lib().qevict_create(C.byref(cfg), device_mem_ptr, n_bytes, C.byref(h)))
    return h


def qevict_destroy(h):
    _check(lib().qevict_destroy(h))


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def qevict_prefill_assign(h, layer, k, v, ctx_tokens, window_scores, stream=None):
    _check(lib().qevict_prefill_assign(h, layer, _ptr(k), _ptr(v), ctx_tokens, _ptr(window_scores), _stream(stream)), h)


def qevict_decode_attn(h, layer, q, k_new, v_new, out, stream=None):
    _check(lib().qevict_decode_attn(h, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _stream(stream)), h)


def qevict_decode_attn_host(h, layer, q, k_new, v_new, out, stream=None):
    """q, k_new, v_new, out: HOST tensors (pinned or pageable)."""
    _check(lib().qevict_decode_attn_host(h, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _stream(stream)), h)


def qevict_decode_attn_host_async(h, layer, q, k_new, v_new, out, stream=None):
    """Host tensors (pinned); the caller synchronises the stream before reading `out`."""
    _check(lib().qevict_decode_attn_host_async(h, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _stream(stream)), h)


def qevict_decode_attn_noalloc(h, layer, q, k_new, v_new, out, stream=None):
    """qevict_decode_attn with the attention scratch in the library's built-in device array: for callers
    that must not allocate device memory.  Raises QEvictError(NO_MEMORY) if the call's scratch does not fit."""
    _check(lib().qevict_decode_attn_noalloc(h, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _stream(stream)), h)


def qevict_wait_result(h):
    """Blocks until the result of the last qevict_decode_attn_host_async call is in host memory."""
    _check(lib().qevict_wait_result(h), h)


def qevict_rebalance(h, layer, stream=None):
    _check(lib().qevict_rebalance(h, layer, _stream(stream)), h)


def qevict_state_layout_of(h):
    lay = qevict_state_layout()
    _check(lib().qevict_state_layout_of(h, C.byref(lay)), h)
    return lay


def _state_buffers(lay):
    """Host tensors of a snapshot, sized by the layout."""
    nw, i32, f32, u8 = lay.n_window_slots, torch.int32, torch.float32, torch.uint8
    return {
        "tier": torch.zeros(nw, dtype=u8), "ledger": torch.zeros(nw, dtype=u8),
        "fp_page": torch.zeros(nw, dtype=i32), "q_page": torch.zeros(nw, dtype=i32),
        "importance": torch.zeros(nw, dtype=f32), "event_mass": torch.zeros(nw, dtype=f32),
        "fp_owner": torch.zeros(lay.n_fp_pages, dtype=i32), "q_owner": torch.zeros(lay.n_q_pages, dtype=i32),
        "entries": torch.zeros((lay.n_entries, 2), dtype=i32), "last_mass": torch.zeros(lay.n_entries, dtype=f32),
        "fp_pool": torch.zeros(lay.fp_pool_bytes, dtype=u8), "q_pool": torch.zeros(lay.q_pool_bytes, dtype=u8),
    }


def _state_view(arrays):
    view = qevict_state_view()
    view.struct_size = C.sizeof(qevict_state_view)
    for n in _STATE_ARRAYS:
        t = arrays[n]
        assert not t.is_cuda and t.is_contiguous()
        setattr(view, n, t.data_ptr())
    return view


def qevict_export_state(h, layer, seq):
    """Snapshot of one unit: a dict of host tensors (tables, owner tables, work list, the unit's pages of both pools
    in the library's page layout) and scalars.  Synchronises."""
    arrays = _state_buffers(qevict_state_layout_of(h))
    view = _state_view(arrays)
    _check(lib().qevict_export_state(h, layer, seq, C.byref(view)), h)
    state = dict(arrays)
    for n in _STATE_SCALARS:
        state[n] = int(getattr(view, n))
    state["knorm_acc"] = float(view.knorm_acc)
    state["counters"] = [int(x) for x in view.counters]
    state["decode_steps"] = int(view.decode_steps)
    return state


def qevict_import_state(h, layer, seq, state):
    """Restores a unit from a snapshot made by qevict_export_state on a cache of the same configuration."""
    view = _state_view(state)
    for n in _STATE_SCALARS:
        setattr(view, n, int(state[n]))
    view.knorm_acc = float(state["knorm_acc"])
    for i in range(4):
        view.counters[i] = int(state["counters"][i])
    view.decode_steps = int(state["decode_steps"])
    _check(lib().qevict_import_state(h, layer, seq, C.byref(view)), h)


def qevict_set_splits(h, splits):
    _check(lib().qevict_set_splits(h, splits), h)


def qevict_set_kernel_timing(h, enable):
    _check(lib().qevict_set_kernel_timing(h, int(enable)), h)


def qevict_kernel_time(h):
    ms, n = C.c_double(), C.c_uint64()
    _check(lib().qevict_kernel_time(h, C.byref(ms), C.byref(n)), h)
    return ms.value, n.value


KERNEL_NAMES = ("append", "decode_attn", "combine", "route", "migrate")


def qevict_kernel_times(h):
    ms = (C.c_double * len(KERNEL_NAMES))()
    n = (C.c_uint64 * len(KERNEL_NAMES))()
    _check(lib().qevict_kernel_times(h, ms, n), h)
    return {name: (ms[i], n[i]) for i, name in enumerate(KERNEL_NAMES)}


def qevict_kernel_timeline(h, max_records=2560):
    kid = (C.c_int32 * max_records)()
    t0 = (C.c_double * max_records)()
    t1 = (C.c_double * max_records)()
    n = C.c_int32(0)
    _check(lib().qevict_kernel_timeline(h, max_records, kid, t0, t1, C.byref(n)), h)
    return [(KERNEL_NAMES[kid[i]] if 0 <= kid[i] < len(KERNEL_NAMES) else "k%d" % kid[i], t0[i], t1[i]) for i in range(n.value)]


def qevict_get_stats(h, layer=-1):
    st = qevict_stats()
    _check(lib().qevict_get_stats(h, layer, C.byref(st)), h)
    return {n: getattr(st, n) for n, _ in qevict_stats._fields_}


def qevict_check_device(h):
    """Synchronises; raises QEvictError(DEVICE_CHECK) if a kernel recorded a failed check, else returns 0."""
    code = C.c_int32(0)
    _check(lib().qevict_check_device(h, C.byref(code)), h)
    return code.value


def qevict_launch_count(h):
    return lib().qevict_launch_count(h)


class QEvictCache:
    """A cache handle together with the torch-allocated device workspace it lives in."""

    def __init__(self, cfg):
        self.cfg = cfg
        self.device = torch.device("cuda", cfg.device)
        self.torch_dtype = torch.float16 if cfg.dtype == DTYPE_FP16 else torch.bfloat16
        self.n_bytes = qevict_workspace_bytes(cfg)
        self.workspace = torch.empty(self.n_bytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        self.handle = qevict_create(cfg, C.c_void_p(base), self.n_bytes)
        self.max_windows = cfg.max_context // cfg.window

    def close(self):
        if self.handle is not None:
            torch.cuda.synchronize(self.device)
            qevict_destroy(self.handle)
            self.handle = None
            self.workspace = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the hot path -----------------------------------------------------------------------------
    def prefill_assign(self, layer, k, v, window_scores, stream=None):
        assert k.is_cuda and k.is_contiguous() and v.is_contiguous() and k.dtype == self.torch_dtype
        assert window_scores.dtype == torch.float32 and window_scores.is_contiguous()
        qevict_prefill_assign(self.handle, layer, k, v, k.shape[-2], window_scores, stream)

    def prefill_score(self, k, q_obs, stream=None):
        """k [batch, H_kv, ctx, d], q_obs [batch, n_obs, H_q, d] (device) -> window scores [batch, ctx / W] float32."""
        n_obs, ctx = q_obs.shape[1], k.shape[-2]
        need = C.c_uint64()
        _check(lib().qevict_prefill_score_scratch_bytes(self.handle, n_obs, ctx, C.byref(need)), self.handle)
        scratch = torch.empty(need.value, dtype=torch.uint8, device=self.device)
        scores = torch.empty((k.shape[0], ctx // self.cfg.window), dtype=torch.float32, device=self.device)
        _check(lib().qevict_prefill_score(self.handle, _ptr(k), _ptr(q_obs), n_obs, ctx, _ptr(scores), _ptr(scratch),
                                          need.value, _stream(stream)), self.handle)
        return scores

    def decode_attn(self, layer, q, k_new=None, v_new=None, out=None, stream=None):
        assert q.is_cuda and q.is_contiguous() and q.dtype == self.torch_dtype
        if out is None:
            out = torch.empty_like(q)
        qevict_decode_attn(self.handle, layer, q, k_new, v_new, out, stream)
        return out

    def decode_attn_host(self, layer, q, k_new, v_new, out, stream=None):
        qevict_decode_attn_host(self.handle, layer, q, k_new, v_new, out, stream)
        return out

    def decode_attn_host_async(self, layer, q, k_new, v_new, out, stream=None):
        qevict_decode_attn_host_async(self.handle, layer, q, k_new, v_new, out, stream)

    def wait_result(self):
        qevict_wait_result(self.handle)

    def rebalance(self, layer, stream=None):
        qevict_rebalance(self.handle, layer, stream)

    def set_splits(self, splits):
        qevict_set_splits(self.handle, splits)

    def set_kernel_timing(self, enable):
        qevict_set_kernel_timing(self.handle, enable)

    def kernel_time(self):
        """(summed milliseconds, launches) of the attention kernel since the last call."""
        return qevict_kernel_time(self.handle)

    def kernel_times(self):
        """{kernel name: (summed milliseconds, launches)} since the last call."""
        return qevict_kernel_times(self.handle)

    def kernel_timeline(self, max_records=2560):
        """[(kernel name, start, end)] of the launches since the last call (first 512 API calls), oldest first, in
        microseconds from the first start; tracing library only (QEVICT_TRACE_LIB=1)."""
        return qevict_kernel_timeline(self.handle, max_records)

    def stats(self, layer=-1):
        return qevict_get_stats(self.handle, layer)

    def launch_count(self):
        return qevict_launch_count(self.handle)

    def check_device(self):
        return qevict_check_device(self.handle)

    # -- exports (parity checks, snapshots) -------------------------------------------------------
    def export_state(self, layer, seq):
        return qevict_export_state(self.handle, layer, seq)

    def import_state(self, layer, seq, state):
        qevict_import_state(self.handle, layer, seq, state)

    def export_tables(self, layer, seq):
        n = self.max_windows
        dev = self.device
        out = {
            "n_windows": torch.zeros(1, dtype=torch.int32, device=dev),
            "tier": torch.zeros(n, dtype=torch.uint8, device=dev),
            "ledger": torch.zeros(n, dtype=torch.uint8, device=dev),
            "fp_page": torch.zeros(n, dtype=torch.int32, device=dev),
            "q_page": torch.zeros(n, dtype=torch.int32, device=dev),
            "importance": torch.zeros(n, dtype=torch.float32, device=dev),
        }
        _check(lib().qevict_export_tables(self.handle, layer, seq, _ptr(out["n_windows"]), _ptr(out["tier"]),
                                          _ptr(out["ledger"]), _ptr(out["fp_page"]), _ptr(out["q_page"]),
                                          _ptr(out["importance"]), _stream(None)), self.handle)
        return {k: v.cpu() for k, v in out.items()}

    def export_last_mass(self, layer, seq):
        m = torch.zeros(self.max_windows, dtype=torch.float32, device=self.device)
        _check(lib().qevict_export_last_mass(self.handle, layer, seq, _ptr(m), _stream(None)), self.handle)
        return m.cpu()

    def export_event_mass(self, layer, seq):
        m = torch.zeros(self.max_windows, dtype=torch.float32, device=self.device)
        _check(lib().qevict_export_event_mass(self.handle, layer, seq, _ptr(m), _stream(None)), self.handle)
        return m.cpu()

    def export_fp_page(self, layer, seq, page):
        c = self.cfg
        k = torch.empty((c.n_kv_heads, c.window, c.head_dim), dtype=self.torch_dtype, device=self.device)
        v = torch.empty_like(k)
        _check(lib().qevict_export_fp_page(self.handle, layer, seq, page, _ptr(k), _ptr(v), _stream(None)), self.handle)
        return k.cpu(), v.cpu()

    def export_q_page(self, layer, seq, page):
        c = self.cfg
        g = c.group_size
        kc = torch.empty((c.n_kv_heads, c.window, c.head_dim), dtype=torch.uint8, device=self.device)
        vc = torch.empty_like(kc)
        kp = torch.empty((c.n_kv_heads, c.window // g, c.head_dim, 2), dtype=self.torch_dtype, device=self.device)
        vp = torch.empty((c.n_kv_heads, c.window, c.head_dim // g, 2), dtype=self.torch_dtype, device=self.device)
        _check(lib().qevict_export_q_page(self.handle, layer, seq, page, _ptr(kc), _ptr(kp), _ptr(vc), _ptr(vp),
                                          _stream(None)), self.handle)
        return kc.cpu(), kp.cpu(), vc.cpu(), vp.cpu()
