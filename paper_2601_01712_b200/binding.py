"""ctypes binding of ``librelaygr.so``: same names as ``include/relaygr.h``, argument
marshalling only.  Pointers are plain integers (``tensor.data_ptr()``), numpy host
arrays, or ``None``.  The library must have been built (``build.build()``); there
is no fallback of any kind when it is missing."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librelaygr.so")

OK, E_INVALID, E_NOSPACE, E_EXISTS, E_MISS, E_BUSY, E_CUDA, E_UNSUPPORTED = 0, -1, -2, -3, -4, -5, -6, -7
DTYPE_F32, DTYPE_BF16 = 0, 1
TIER_MISS, TIER_ALLOCATED, TIER_HBM, TIER_LOADING, TIER_HOST = 0, 1, 2, 3, 4
DEVSTATUS_WAIT_TIMEOUT, DEVSTATUS_BAD_INDEX = 1, 2      # RELAYGR_DEVSTATUS_*: codes of the device status word

STATUS_NAMES = {0: "OK", -1: "E_INVALID", -2: "E_NOSPACE", -3: "E_EXISTS", -4: "E_MISS", -5: "E_BUSY", -6: "E_CUDA",
                -7: "E_UNSUPPORTED"}


class ModelCfg(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32), ("d_head", C.c_int32),
                ("d_ff", C.c_int32), ("dtype", C.c_int32), ("page_tokens", C.c_int32), ("vocab", C.c_int64),
                ("ln_eps", C.c_float), ("attn_kind", C.c_int32)]


WEIGHT_FIELDS = ["emb", "ln1_g", "ln1_b", "ln2_g", "ln2_b", "w_qkv", "b_qkv", "w_o", "b_o", "w1", "b1", "w2", "b2",
                 "lnf_g", "lnf_b", "w_score", "b_score"]


class Weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in WEIGHT_FIELDS]


class PoolStats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in
                ["pages_total", "pages_free", "host_pages_total", "host_pages_free", "users_hbm", "users_loading",
                 "users_host", "users_allocated", "hits_hbm", "hits_loading", "hits_host", "misses", "reloads",
                 "reload_bytes", "spills", "spill_bytes"]]

    def as_dict(self):
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


class Profile(C.Structure):
    _fields_ = [(n, C.c_double) for n in ["gather_ln_ms", "layernorm_ms", "gemm_ms", "attention_ms", "score_ms"]] + \
               [(n, C.c_int64) for n in ["gather_ln_launches", "layernorm_launches", "gemm_launches",
                                         "attention_launches", "score_launches"]]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class RelayGRError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("%s: %s" % (STATUS_NAMES.get(code, code), msg))
        self.code = code


# every symbol include/relaygr.h declares: name -> (restype, argtypes)
_P, _I32, _I64, _U64, _SZ = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_size_t
SIGNATURES = {
    "relaygr_create": (_I32, [C.POINTER(ModelCfg), C.POINTER(Weights), C.POINTER(_P)]),
    "relaygr_create_host_only": (_I32, [C.POINTER(ModelCfg), C.POINTER(_P)]),
    "relaygr_destroy": (_I32, [_P]),
    "relaygr_last_error": (C.c_char_p, []),
    "relaygr_workspace_bytes": (_I32, [_P, _I64, _I64, _I64, C.POINTER(_SZ)]),
    "relaygr_set_workspace": (_I32, [_P, _P, _SZ]),
    "relaygr_device_status": (_I32, [_P, _P, C.POINTER(_I32)]),
    "relaygr_attention_plan": (_I32, [_I32, _I32, _P, _P, _P, _I32, _I32, _P, _I32, C.POINTER(_I32), _P, _I32, C.POINTER(_I32)]),
    "relaygr_kv_page_bytes": (_I32, [_P, C.POINTER(_SZ)]),
    "relaygr_kv_pool_create": (_I32, [_P, _P, _SZ, _P, _SZ, C.POINTER(_P)]),
    "relaygr_kv_pool_destroy": (_I32, [_P]),
    "relaygr_kv_set_max_inflight_reloads": (_I32, [_P, _I32]),
    "relaygr_kv_alloc": (_I32, [_P, _U64, _I32, _P]),
    "relaygr_kv_commit": (_I32, [_P, _U64, _P]),
    "relaygr_kv_wait_pages": (_I32, [_P, _U64, _P]),
    "relaygr_kv_host_backend_control": (_I32, [_P, _I32, _I64, C.POINTER(_I64)]),
    "relaygr_kv_free": (_I32, [_P, _U64]),
    "relaygr_kv_evict": (_I32, [_P, _U64, _I32, _P]),
    "relaygr_kv_reload_from_host": (_I32, [_P, _U64, _P, C.POINTER(_P)]),
    "relaygr_kv_lookup": (_I32, [_P, _U64, C.POINTER(_I32), C.POINTER(_I32)]),
    "relaygr_kv_pages": (_I32, [_P, _U64, _P, _I32, C.POINTER(_I32)]),
    "relaygr_kv_stats": (_I32, [_P, C.POINTER(PoolStats)]),
    "relaygr_gather": (_I32, [_P, _P, _I64, _P, _P]),
    "relaygr_preinfer": (_I32, [_P, _P, _I32, _P, _P, _P, _P]),
    "relaygr_rank": (_I32, [_P, _P, _I32, _P, _P, _P, _P, _P, _P, _P, _P]),
    "relaygr_rank_full": (_I32, [_P, _I32, _P, _P, _P, _P, _P, _P, _P, _P]),
    "relaygr_rank_full_static": (_I32, [_P, _I32, _P, _P, _P, _P, _P, _P, _P, _P]),
    "relaygr_profile_enable": (_I32, [_P, _I32]),
    "relaygr_profile_read": (_I32, [_P, C.POINTER(Profile)]),
    "relaygr_launch_count": (_I32, [_P, C.POINTER(_I64)]),
}

_lib = None


def lib():
    """The loaded library.  Raises if it has not been built: there is no other path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("librelaygr.so is missing: run paper_2601_01712_b200.build.build() "
                               "(or __graft_entry__.build()); this package has no CPU or PyTorch fallback")
        l = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype, fn.argtypes = res, args
        _lib = l
    return _lib


def last_error() -> str:
    return lib().relaygr_last_error().decode()


def _check(code, ok=(OK,)):
    if code not in ok:
        raise RelayGRError(code, last_error())
    return code


def _ptr(x):
    """int / None / numpy array / torch tensor -> address."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        assert x.flags["C_CONTIGUOUS"]
        return x.ctypes.data
    return x.data_ptr()


def _host_i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a


def _host_u64(a):
    return np.ascontiguousarray(a, dtype=np.uint64)


def relaygr_create(cfg: ModelCfg, weights: Weights) -> int:
    out = _P()
    _check(lib().relaygr_create(C.byref(cfg), C.byref(weights), C.byref(out)))
    return out.value


def relaygr_create_host_only(cfg: ModelCfg) -> int:
    out = _P()
    _check(lib().relaygr_create_host_only(C.byref(cfg), C.byref(out)))
    return out.value


def relaygr_destroy(ctx):
    _check(lib().relaygr_destroy(ctx))


def relaygr_workspace_bytes(ctx, max_rows, max_users, max_pages) -> int:
    out = _SZ()
    _check(lib().relaygr_workspace_bytes(ctx, max_rows, max_users, max_pages, C.byref(out)))
    return out.value


def relaygr_set_workspace(ctx, dev, nbytes):
    _check(lib().relaygr_set_workspace(ctx, _ptr(dev), nbytes))


def relaygr_device_status(ctx, stream=None) -> int:
    out = _I32()
    _check(lib().relaygr_device_status(ctx, stream, C.byref(out)))
    return out.value


def relaygr_attention_plan(mode, prefix_len, short_len, cand_len, n_heads, n_sms):
    """The attention work list of a call (host only).  Returns (items [n, 8], merges [m, 6]) as int32 numpy arrays."""
    import numpy as np
    n = len(prefix_len)
    arr = lambda v: np.ascontiguousarray(np.asarray(v if v is not None else [0] * n, dtype=np.int32))
    p, s_, c_ = arr(prefix_len), arr(short_len), arr(cand_len)
    n_items, n_merges = _I32(), _I32()
    cap_i, cap_m = 4096, 1024
    while True:
        items = np.zeros((cap_i, 8), dtype=np.int32)
        merges = np.zeros((cap_m, 6), dtype=np.int32)
        rc = lib().relaygr_attention_plan(mode, n, p.ctypes.data, s_.ctypes.data, c_.ctypes.data, n_heads, n_sms, items.ctypes.data, cap_i,
                                          C.byref(n_items), merges.ctypes.data, cap_m, C.byref(n_merges))
        if rc == E_NOSPACE:
            cap_i, cap_m = max(cap_i, n_items.value), max(cap_m, n_merges.value)
            continue
        _check(rc)
        return items[:n_items.value].copy(), merges[:n_merges.value].copy()


def relaygr_kv_page_bytes(ctx) -> int:
    out = _SZ()
    _check(lib().relaygr_kv_page_bytes(ctx, C.byref(out)))
    return out.value


def relaygr_kv_pool_create(ctx, hbm_slab, hbm_bytes, host_slab=None, host_bytes=0) -> int:
    out = _P()
    _check(lib().relaygr_kv_pool_create(ctx, _ptr(hbm_slab), hbm_bytes, _ptr(host_slab), host_bytes, C.byref(out)))
    return out.value


def relaygr_kv_pool_destroy(pool):
    _check(lib().relaygr_kv_pool_destroy(pool))


def relaygr_kv_set_max_inflight_reloads(pool, n):
    _check(lib().relaygr_kv_set_max_inflight_reloads(pool, n))


def relaygr_kv_alloc(pool, user, prefix_len, page_ids=None, ok=(OK,)) -> int:
    ids = None if page_ids is None else _host_i32(page_ids)
    return _check(lib().relaygr_kv_alloc(pool, user, prefix_len, _ptr(ids)), ok)


def relaygr_kv_commit(pool, user, stream=None, ok=(OK,)) -> int:
    return _check(lib().relaygr_kv_commit(pool, user, stream), ok)


def relaygr_kv_wait_pages(pool, user, stream=None, ok=(OK,)) -> int:
    return _check(lib().relaygr_kv_wait_pages(pool, user, stream), ok)


HOSTCTL_MANUAL_EVENTS, HOSTCTL_COMPLETE_EVENTS, HOSTCTL_FAIL_COPIES, HOSTCTL_STREAM_WAITS, HOSTCTL_PENDING_EVENTS = range(5)


def relaygr_kv_host_backend_control(pool, what, arg=0, ok=(OK,)):
    """Returns (status, value) of a test-control request to a host-only pool."""
    out = _I64(0)
    code = _check(lib().relaygr_kv_host_backend_control(pool, what, arg, C.byref(out)), ok)
    return code, out.value


def relaygr_kv_free(pool, user, ok=(OK,)) -> int:
    return _check(lib().relaygr_kv_free(pool, user), ok)


def relaygr_kv_evict(pool, user, spill_to_host, side_stream=None, ok=(OK,)) -> int:
    return _check(lib().relaygr_kv_evict(pool, user, int(spill_to_host), side_stream), ok)


def relaygr_kv_reload_from_host(pool, user, side_stream=None, ok=(OK,)):
    """Returns (status, ready_event or None)."""
    ev = _P()
    code = _check(lib().relaygr_kv_reload_from_host(pool, user, side_stream, C.byref(ev)), ok)
    return code, ev.value


def relaygr_kv_lookup(pool, user):
    """Returns (tier, prefix_len)."""
    tier, plen = _I32(), _I32()
    _check(lib().relaygr_kv_lookup(pool, user, C.byref(tier), C.byref(plen)))
    return tier.value, plen.value


def relaygr_kv_pages(pool, user) -> np.ndarray:
    n = _I32()
    _check(lib().relaygr_kv_pages(pool, user, None, 0, C.byref(n)))
    out = np.zeros(n.value, dtype=np.int32)
    _check(lib().relaygr_kv_pages(pool, user, _ptr(out), n.value, C.byref(n)))
    return out


def relaygr_kv_stats(pool) -> dict:
    st = PoolStats()
    _check(lib().relaygr_kv_stats(pool, C.byref(st)))
    return st.as_dict()


def relaygr_gather(ctx, ids_dev, n, out_dev, stream=None):
    _check(lib().relaygr_gather(ctx, _ptr(ids_dev), n, _ptr(out_dev), stream))


def relaygr_preinfer(ctx, pool, users, prefix_ids_dev, prefix_off, stream=None, ok=(OK,)) -> int:
    users, off = _host_u64(users), _host_i32(prefix_off)
    return _check(lib().relaygr_preinfer(ctx, pool, len(users), _ptr(users), _ptr(prefix_ids_dev), _ptr(off), stream), ok)


def relaygr_rank(ctx, pool, users, short_ids_dev, short_off, cand_ids_dev, cand_off, scores_dev, stream=None,
                 per_user_status=None, ok=(OK,)) -> int:
    users, so, co = _host_u64(users), _host_i32(short_off), _host_i32(cand_off)
    return _check(lib().relaygr_rank(ctx, pool, len(users), _ptr(users), _ptr(short_ids_dev), _ptr(so),
                                     _ptr(cand_ids_dev), _ptr(co), _ptr(scores_dev), _ptr(per_user_status), stream), ok)


def relaygr_rank_full(ctx, n_users, prefix_ids_dev, prefix_off, short_ids_dev, short_off, cand_ids_dev, cand_off,
                      scores_dev, stream=None, ok=(OK,)) -> int:
    po, so, co = _host_i32(prefix_off), _host_i32(short_off), _host_i32(cand_off)
    return _check(lib().relaygr_rank_full(ctx, n_users, _ptr(prefix_ids_dev), _ptr(po), _ptr(short_ids_dev), _ptr(so),
                                          _ptr(cand_ids_dev), _ptr(co), _ptr(scores_dev), stream), ok)


STATIC_SCRATCH_BYTES = 96 << 20      # RELAYGR_STATIC_SCRATCH_BYTES


def relaygr_rank_full_static(ctx, n_users, prefix_ids_dev, prefix_off, short_ids_dev, short_off, cand_ids_dev, cand_off,
                             scores_dev, stream=None, ok=(OK,)) -> int:
    """Full inference on the scratch array built into the library: for callers that may not allocate device
    memory and have no workspace to lend.  Batches beyond the array's size return E_NOSPACE."""
    po, so, co = _host_i32(prefix_off), _host_i32(short_off), _host_i32(cand_off)
    return _check(lib().relaygr_rank_full_static(ctx, n_users, _ptr(prefix_ids_dev), _ptr(po), _ptr(short_ids_dev), _ptr(so),
                                                 _ptr(cand_ids_dev), _ptr(co), _ptr(scores_dev), stream), ok)


def relaygr_profile_enable(ctx, on: bool):
    _check(lib().relaygr_profile_enable(ctx, int(on)))


def relaygr_profile_read(ctx) -> dict:
    out = Profile()
    _check(lib().relaygr_profile_read(ctx, C.byref(out)))
    return out.as_dict()


def relaygr_launch_count(ctx) -> int:
    out = _I64()
    _check(lib().relaygr_launch_count(ctx, C.byref(out)))
    return out.value
