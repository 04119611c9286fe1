"""numpy front end of the CPU oracle (test infrastructure only).

Only the tests, the smoke check and the CPU-baseline leg of the benchmark may
import this package; the GPU library never does.  Arrays are dense and
C-contiguous, laid out [B, L, H, T_cap, D]; bfloat16 data travels as uint16
bit patterns (``dtype='bf16'``), fp32 as float32.

The ``*_packed`` forms take ragged caches without padding: tensors [H, total_rows, D]
(index map and keys [H, total_rows]) plus ``rows = (row_off, row_cap, total_rows)``,
where the rows of (b, l) are [row_off[b, l], row_off[b, l] + row_cap[b, l]) for every
head.  They compute what the dense forms compute; only the addressing differs.
"""
import ctypes
import os

import numpy as np

from . import build as _build

_DT = {"f32": 0, "bf16": 1}
_LIB = None


def lib():
    global _LIB
    if _LIB is None:
        _LIB = ctypes.CDLL(_build.build())
        _LIB.l2kv_oracle_keep_count.restype = ctypes.c_int32
        _LIB.l2kv_oracle_keep_count.argtypes = [ctypes.c_int32, ctypes.c_double]
    return _LIB


def _p(a):
    return ctypes.c_void_p(a.ctypes.data)


def _check(a, dtype):
    want = np.uint16 if dtype == "bf16" else np.float32
    if a.dtype != want or not a.flags["C_CONTIGUOUS"]:
        raise ValueError(f"expected contiguous {want} for dtype {dtype}, got {a.dtype}")


def _i32(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.int32))


def hardware_threads():
    return int(lib().l2kv_oracle_hardware_threads())


def keep_count(length, keep_ratio):
    return int(lib().l2kv_oracle_keep_count(int(length), float(keep_ratio)))


def key_sumsq(K, dtype):
    """fp64 sum of squares of every row of K[..., D]."""
    _check(K, dtype)
    D = K.shape[-1]
    out = np.empty(K.shape[:-1], dtype=np.float64)
    lib().l2kv_oracle_key_sumsq(_p(K), _DT[dtype], ctypes.c_int64(out.size), D, _p(out))
    return out


def key_sumsq_f32(K, dtype):
    """Sum of squares in the GPU library's documented fp32 summation order."""
    _check(K, dtype)
    D = K.shape[-1]
    out = np.empty(K.shape[:-1], dtype=np.float32)
    lib().l2kv_oracle_key_sumsq_f32(_p(K), _DT[dtype], ctypes.c_int64(out.size), D, _p(out))
    return out


def select(key, keep, policy=0):
    """Positions (ascending) of the `keep` lowest keys of a 1-D float64 array."""
    key = np.ascontiguousarray(key, dtype=np.float64)
    out = np.empty(keep, dtype=np.int32)
    lib().l2kv_oracle_select(_p(key), int(key.size), int(keep), int(policy), _p(out))
    return out


def random_key(seed, unit, t):
    """Ordering key of the keep-random policy for token t of unit (b * L + l) * H + h."""
    f = lib().l2kv_oracle_random_key
    f.restype = ctypes.c_uint32
    f.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint32]
    return int(f(seed & 0xFFFFFFFFFFFFFFFF, unit, t))


def compress(K, V, dtype, lens, keep, uncompressed=(), key_mode=0, policy=0, t_cap_out=None,
             nthreads=1, seed=0):
    """Whole-cache compression.  Returns dict(K_c, V_c, idx, key, kept_len).  `keep` is [B],
    or [B, L, H] for a keep count per head; kept_len is then [B, L, H] too."""
    _check(K, dtype)
    _check(V, dtype)
    B, L, H, T_cap, D = K.shape
    lens, keep, unc = _i32(lens), _i32(keep), _i32(list(uncompressed))
    per_head = keep.ndim == 3
    if per_head:
        assert keep.shape == (B, L, H)
        keep_unit, keep = keep, np.zeros(B, dtype=np.int32)
        kept_len_unit = np.zeros((B, L, H), dtype=np.int32)
    if t_cap_out is None:
        t_cap_out = T_cap
    K_c = np.zeros((B, L, H, t_cap_out, D), dtype=K.dtype)
    V_c = np.zeros_like(K_c)
    idx = np.full((B, L, H, t_cap_out), -1, dtype=np.int32)
    key = np.full((B, L, H, t_cap_out), np.nan, dtype=np.float64)
    kept_len = np.zeros((B, L), dtype=np.int32)
    rc = lib().l2kv_oracle_compress(
        _p(K), _p(V), _DT[dtype], B, L, H, T_cap, D, _p(lens), _p(keep), _p(unc), int(unc.size),
        int(key_mode), int(policy), ctypes.c_uint64(int(seed) & 0xFFFFFFFFFFFFFFFF), int(t_cap_out),
        _p(K_c), _p(V_c), _p(idx), _p(key),
        _p(kept_len), _p(keep_unit) if per_head else None,
        _p(kept_len_unit) if per_head else None, int(nthreads))
    if rc != 0:
        raise ValueError(f"oracle compress: bad argument ({rc})")
    return dict(K_c=K_c, V_c=V_c, idx=idx, key=key,
                kept_len=kept_len_unit if per_head else kept_len)


def attention(q, K_c, V_c, dtype, cur_len, scale=0.0, nthreads=1):
    """Decode attention, fp64 two-pass softmax.  q [B, L, Hq, D] -> float64 [B, L, Hq, D].
    cur_len is [B, L], or [B, L, Hkv] for a length per KV head."""
    _check(q, dtype)
    _check(K_c, dtype)
    _check(V_c, dtype)
    B, L, Hkv, T_cap, D = K_c.shape
    Hq = q.shape[2]
    cur_len = _i32(cur_len)
    per_head = cur_len.ndim == 3
    if per_head:
        cur_len_unit, cur_len = cur_len.reshape(B, L, Hkv), np.zeros((B, L), dtype=np.int32)
    else:
        cur_len = cur_len.reshape(B, L)
    out = np.empty((B, L, Hq, D), dtype=np.float64)
    rc = lib().l2kv_oracle_attention(
        _p(q), _p(K_c), _p(V_c), _DT[dtype], B, L, Hkv, Hq, T_cap, D, _p(cur_len),
        ctypes.c_double(scale), _p(out), _p(cur_len_unit) if per_head else None, int(nthreads))
    if rc != 0:
        raise ValueError(f"oracle attention: bad argument ({rc})")
    return out


def append_evict(state, dtype, budget, uncompressed, k_new, v_new, pos_new, key_mode=0):
    """One append/evict step, in place on state = dict(K_c, V_c, idx, key, cur_len).

    cur_len [B, L] with budget [B], or (a length and a budget per head) both [B, L, H].
    Returns the oracle's status (0, or -2 when a row did not fit T_cap).
    """
    K_c, V_c = state["K_c"], state["V_c"]
    _check(K_c, dtype)
    _check(k_new, dtype)
    _check(v_new, dtype)
    B, L, H, T_cap, D = K_c.shape
    budget, unc, pos_new = _i32(budget), _i32(list(uncompressed)), _i32(pos_new)
    assert state["idx"].dtype == np.int32 and state["key"].dtype == np.float64
    per_head = state["cur_len"].ndim == 3
    assert state["cur_len"].dtype == np.int32
    assert state["cur_len"].shape == ((B, L, H) if per_head else (B, L))
    assert budget.shape == ((B, L, H) if per_head else (B,))
    return int(lib().l2kv_oracle_append_evict(
        _p(K_c), _p(V_c), _p(state["idx"]), _p(state["key"]), _DT[dtype], B, L, H, T_cap, D,
        _p(state["cur_len"]), _p(budget), _p(unc), int(unc.size), _p(k_new), _p(v_new),
        _p(pos_new), int(key_mode), int(per_head)))


def attention_loss(q, K, dtype, cur_len, scale=0.0, key_mode=0, curves=False, nthreads=1):
    """Attention loss of norm-based vs ideal compression (Eqs. 5-7).  Returns alr [B, L, Hq]
    (float64) and, with curves=True, also (loss, loss_ref) [B, L, Hq, T_cap] (NaN past n)."""
    _check(q, dtype)
    _check(K, dtype)
    B, L, Hkv, T_cap, D = K.shape
    Hq = q.shape[2]
    cur_len = _i32(cur_len).reshape(B, L)
    alr = np.zeros((B, L, Hq), dtype=np.float64)
    loss = np.full((B, L, Hq, T_cap), np.nan) if curves else None
    ref = np.full((B, L, Hq, T_cap), np.nan) if curves else None
    rc = lib().l2kv_oracle_attention_loss(
        _p(q), _p(K), _DT[dtype], B, L, Hkv, Hq, T_cap, D, _p(cur_len), ctypes.c_double(scale),
        int(key_mode), _p(alr), _p(loss) if curves else None, _p(ref) if curves else None,
        int(nthreads))
    if rc != 0:
        raise ValueError(f"oracle attention_loss: bad argument ({rc})")
    return (alr, loss, ref) if curves else alr


def _rows(rows, B, L):
    off, cap, total = rows
    off = np.ascontiguousarray(np.asarray(off, dtype=np.int64)).reshape(B, L)
    cap = np.ascontiguousarray(np.asarray(cap, dtype=np.int32)).reshape(B, L)
    assert int((off + cap).max()) <= int(total) and int(off.min()) >= 0
    return off, cap, int(total)


def compress_packed(K, V, dtype, in_rows, lens, keep, uncompressed, out_rows, L, key_mode=0,
                    policy=0, nthreads=1, seed=0):
    """compress() on packed tensors K, V [H, total_in, D]; `keep` is [B].  Returns dict(K_c, V_c
    [H, total_out, D], idx, key [H, total_out], kept_len [B, L])."""
    _check(K, dtype)
    _check(V, dtype)
    H, total_in, D = K.shape
    lens, keep, unc = _i32(lens), _i32(keep), _i32(list(uncompressed))
    B = lens.size
    ioff, icap, itot = _rows(in_rows, B, L)
    ooff, ocap, otot = _rows(out_rows, B, L)
    assert itot == total_in
    K_c = np.zeros((H, otot, D), dtype=K.dtype)
    V_c = np.zeros_like(K_c)
    idx = np.full((H, otot), -1, dtype=np.int32)
    key = np.full((H, otot), np.nan, dtype=np.float64)
    kept_len = np.zeros((B, L), dtype=np.int32)
    rc = lib().l2kv_oracle_compress_packed(
        _p(K), _p(V), _DT[dtype], B, L, H, _p(ioff), _p(icap), ctypes.c_int64(itot), D, _p(lens),
        _p(keep), _p(unc), int(unc.size), int(key_mode), int(policy),
        ctypes.c_uint64(int(seed) & 0xFFFFFFFFFFFFFFFF), _p(ooff), _p(ocap), ctypes.c_int64(otot),
        _p(K_c), _p(V_c), _p(idx), _p(key), _p(kept_len), None, None, int(nthreads))
    if rc != 0:
        raise ValueError(f"oracle compress_packed: bad argument ({rc})")
    return dict(K_c=K_c, V_c=V_c, idx=idx, key=key, kept_len=kept_len)


def attention_packed(q, K_c, V_c, dtype, rows, cur_len, scale=0.0, nthreads=1):
    """attention() over a packed cache K_c, V_c [Hkv, total_rows, D]; cur_len [B, L]."""
    _check(q, dtype)
    _check(K_c, dtype)
    _check(V_c, dtype)
    B, L, Hq, D = q.shape
    Hkv = K_c.shape[0]
    off, cap, tot = _rows(rows, B, L)
    assert tot == K_c.shape[1]
    cur_len = _i32(cur_len).reshape(B, L)
    out = np.empty((B, L, Hq, D), dtype=np.float64)
    rc = lib().l2kv_oracle_attention_packed(
        _p(q), _p(K_c), _p(V_c), _DT[dtype], B, L, Hkv, Hq, _p(off), _p(cap), ctypes.c_int64(tot),
        D, _p(cur_len), ctypes.c_double(scale), _p(out), None, int(nthreads))
    if rc != 0:
        raise ValueError(f"oracle attention_packed: bad argument ({rc})")
    return out


def append_evict_packed(state, dtype, rows, budget, uncompressed, k_new, v_new, pos_new, key_mode=0):
    """append_evict() in place on a packed state = dict(K_c, V_c [H, total_rows, D], idx, key
    [H, total_rows], cur_len [B, L]); budget [B]."""
    K_c, V_c = state["K_c"], state["V_c"]
    _check(K_c, dtype)
    _check(k_new, dtype)
    _check(v_new, dtype)
    B, L, H, D = k_new.shape
    off, cap, tot = _rows(rows, B, L)
    assert K_c.shape == (H, tot, D) and state["idx"].shape == (H, tot)
    budget, unc, pos_new = _i32(budget), _i32(list(uncompressed)), _i32(pos_new)
    assert state["idx"].dtype == np.int32 and state["key"].dtype == np.float64
    assert state["cur_len"].dtype == np.int32 and state["cur_len"].shape == (B, L)
    return int(lib().l2kv_oracle_append_evict_packed(
        _p(K_c), _p(V_c), _p(state["idx"]), _p(state["key"]), _DT[dtype], B, L, H, _p(off), _p(cap),
        ctypes.c_int64(tot), D, _p(state["cur_len"]), _p(budget), _p(unc), int(unc.size),
        _p(k_new), _p(v_new), _p(pos_new), int(key_mode), 0))
