"""ctypes binding of libl2kv.so: argument marshalling only."""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# L2KV_LIBRARY selects another build of the same library (a tuning variant).
_LIB_PATH = os.environ.get("L2KV_LIBRARY") or os.path.join(_HERE, "libl2kv.so")
_LIB = None

KEEP_LOWEST_NORM = 0
KEEP_HIGHEST_NORM = 1
KEEP_RANDOM = 2
_DTYPE = {torch.float32: 0, torch.bfloat16: 1}


class L2KVError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class _CLayout(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("layers", ctypes.c_int32),
                ("kv_heads", ctypes.c_int32), ("q_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("t_cap", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("stride_b", ctypes.c_int64), ("stride_l", ctypes.c_int64),
                ("stride_h", ctypes.c_int64), ("stride_t", ctypes.c_int64),
                ("row_off_dev", ctypes.c_void_p), ("row_cap_dev", ctypes.c_void_p),
                ("total_rows", ctypes.c_int64)]


def library_path():
    return _LIB_PATH


def lib():
    """The loaded C library.  Raises if it has not been built: nothing else can run."""
    global _LIB
    if _LIB is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_2406_11430_b200.build` "
                              "(needs nvcc); there is no fallback path")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
        lay = ctypes.POINTER(_CLayout)
        L.l2kv_status_string.restype = ctypes.c_char_p
        L.l2kv_status_string.argtypes = [ctypes.c_int]
        L.l2kv_keep_count.argtypes = [i32, ctypes.c_double, ctypes.POINTER(i32)]
        L.l2kv_workspace_bytes.argtypes = [lay, i32, ctypes.POINTER(sz)]
        L.l2kv_read_device_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
        L.l2kv_key_norms.argtypes = [vp, lay, vp, i32, vp, vp, vp]
        L.l2kv_select_compact.argtypes = [vp, vp, lay, vp, vp, i32, ctypes.POINTER(i32), i32, i32,
                                          ctypes.c_uint64, vp, vp, vp, lay, vp, vp, vp, vp, sz, vp]
        L.l2kv_select_compact_per_head.argtypes = L.l2kv_select_compact.argtypes
        L.l2kv_decode_attention.argtypes = [vp, vp, vp, lay, vp, i32, ctypes.c_float, vp, vp, sz, vp]
        L.l2kv_decode_attention_per_head.argtypes = L.l2kv_decode_attention.argtypes
        L.l2kv_append_evict.argtypes = [vp, vp, vp, vp, lay, vp, vp, ctypes.POINTER(i32), i32,
                                        vp, vp, vp, vp, sz, vp]
        L.l2kv_append_evict_per_head.argtypes = L.l2kv_append_evict.argtypes
        L.l2kv_attention_loss_workspace_bytes.argtypes = [lay, i32, ctypes.POINTER(sz)]
        L.l2kv_attention_loss.argtypes = [vp, vp, lay, vp, i32, ctypes.c_float, vp, vp, vp, vp,
                                          vp, sz, vp]
        L.l2kv_attention_loss_per_head.argtypes = L.l2kv_attention_loss.argtypes
        L.l2kv_prefix_attention.argtypes = [vp, vp, vp, lay, vp, i32, i32, ctypes.c_float, vp, vp,
                                            vp, sz, vp]
        L.l2kv_prefix_attention_per_head.argtypes = L.l2kv_prefix_attention.argtypes
        L.l2kv_prefix_attention_causal.argtypes = L.l2kv_prefix_attention.argtypes
        L.l2kv_prefix_attention_workspace_bytes.argtypes = [lay, i32, i32, ctypes.POINTER(sz)]
        L.l2kv_workspace_reset.argtypes = [vp, sz, lay, vp]
        L.l2kv_selftest_wait_timeout.argtypes = [vp, sz, vp]
        L.l2kv_decode_attention_static_status.argtypes = [vp, ctypes.POINTER(i32), i32]
        L.l2kv_prefix_attention_flags.argtypes = [vp, vp, vp, lay, vp, i32, i32, ctypes.c_float,
                                                  ctypes.c_uint32, vp, vp, vp, sz, vp]
        for name in ("l2kv_prefix_attention", "l2kv_attention_loss_workspace_bytes", "l2kv_attention_loss",
                     "l2kv_keep_count", "l2kv_workspace_bytes", "l2kv_read_device_status",
                     "l2kv_key_norms", "l2kv_select_compact", "l2kv_decode_attention",
                     "l2kv_append_evict", "l2kv_select_compact_per_head",
                     "l2kv_decode_attention_per_head", "l2kv_append_evict_per_head",
                     "l2kv_prefix_attention_per_head", "l2kv_prefix_attention_workspace_bytes",
                     "l2kv_prefix_attention_causal", "l2kv_prefix_attention_flags",
                     "l2kv_workspace_reset", "l2kv_selftest_wait_timeout",
                     "l2kv_decode_attention_static_status", "l2kv_attention_loss_per_head"):
            getattr(L, name).restype = ctypes.c_int
        _LIB = L
    return _LIB


def status_string(status):
    return lib().l2kv_status_string(int(status)).decode()


def _check(rc, where):
    if rc != 0:
        raise L2KVError(rc, where)


class Rows:
    """Row ranges of a packed cache [Hkv, total_rows, D]: the rows of (b, l) are
    [row_off[b, l], row_off[b, l] + row_cap[b, l]) for every head.  Built from host arrays
    [B, L]; holds the device copies the library reads."""

    def __init__(self, row_off, row_cap, total_rows, device):
        import numpy as np
        off = np.ascontiguousarray(np.asarray(row_off, dtype=np.int64))
        cap = np.ascontiguousarray(np.asarray(row_cap, dtype=np.int32))
        if off.ndim != 2 or off.shape != cap.shape:
            raise ValueError("row_off and row_cap must both be [B, L]")
        self.B, self.L = off.shape
        self.total_rows = int(total_rows)
        self.t_cap = int(cap.max()) if cap.size else 0
        self.off = torch.from_numpy(off).to(device)
        self.cap = torch.from_numpy(cap).to(device)


class Layout:
    """Geometry of a cache tensor, taken from the tensor: dense [B, L, Hkv, t_cap, D], or,
    with rows (a Rows), packed [Hkv, total_rows, D].  D contiguous."""

    def __init__(self, cache, q_heads=None, rows=None):
        if cache.dtype not in _DTYPE:
            raise ValueError(f"unsupported dtype {cache.dtype}")
        if rows is not None:
            if cache.dim() != 3 or cache.stride(2) != 1 or cache.shape[1] != rows.total_rows:
                raise ValueError("packed cache must be [Hkv, total_rows, D] with D contiguous")
            H, _, D = cache.shape
            self.c = _CLayout(rows.B, rows.L, H, H if q_heads is None else q_heads, D, rows.t_cap,
                              _DTYPE[cache.dtype], 0, 0, 0, cache.stride(0), cache.stride(1),
                              rows.off.data_ptr(), rows.cap.data_ptr(), rows.total_rows)
            self.rows = rows                      # keeps the device arrays alive
            return
        if cache.dim() != 5 or cache.stride(4) != 1:
            raise ValueError("cache must be [B, L, Hkv, t_cap, D] with D contiguous")
        B, L, H, T, D = cache.shape
        sb, sl, sh, st, _ = cache.stride()
        self.c = _CLayout(B, L, H, H if q_heads is None else q_heads, D, T, _DTYPE[cache.dtype], 0,
                          sb, sl, sh, st, None, None, 0)

    def ref(self):
        return ctypes.byref(self.c)


def _ptr(t):
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


_RAW_STREAM = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream(stream, ref=None):
    """Handle of the CUDA stream a call is ordered on: the given torch stream, else the current
    stream of the device that holds `ref` (a tensor of the call); 0 for host-only calls
    (argument checks on host tensors, or no GPU at all)."""
    if stream is not None:
        return ctypes.c_void_p(stream.cuda_stream)
    if ref is not None:
        if not ref.is_cuda:
            return ctypes.c_void_p(0)
        if _RAW_STREAM is not None:              # the handle without building a Stream object
            return ctypes.c_void_p(_RAW_STREAM(ref.device.index))
        return ctypes.c_void_p(torch.cuda.current_stream(ref.device).cuda_stream)
    if not torch.cuda.is_available():
        return ctypes.c_void_p(0)
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _layers(layers):
    layers = list(layers or ())
    arr = (ctypes.c_int32 * max(1, len(layers)))(*layers)
    return arr, len(layers)


def keep_count(length, keep_ratio):
    out = ctypes.c_int32(0)
    _check(lib().l2kv_keep_count(int(length), float(keep_ratio), ctypes.byref(out)), "l2kv_keep_count")
    return out.value


def workspace_bytes(layout, max_len):
    out = ctypes.c_size_t(0)
    _check(lib().l2kv_workspace_bytes(layout.ref(), int(max_len), ctypes.byref(out)),
           "l2kv_workspace_bytes")
    return out.value


def new_workspace(layout, max_len, device):
    """A zeroed device buffer large enough for any call on this layout."""
    return torch.zeros(workspace_bytes(layout, max_len), dtype=torch.uint8, device=device)


def read_device_status(workspace, stream=None):
    out = ctypes.c_int32(0)
    _check(lib().l2kv_read_device_status(_ptr(workspace), _stream(stream, workspace), ctypes.byref(out)),
           "l2kv_read_device_status")
    return out.value


def workspace_reset(workspace, layout, stream=None):
    """Zeroes the status block and the completion counters of a workspace, in stream order."""
    _check(lib().l2kv_workspace_reset(_ptr(workspace), workspace.numel(), layout.ref(), _stream(stream, workspace)),
           "l2kv_workspace_reset")


def selftest_wait_timeout(workspace, stream=None):
    """Makes one bounded wait run out on purpose (nothing faults) and records it in workspace."""
    _check(lib().l2kv_selftest_wait_timeout(_ptr(workspace), workspace.numel(), _stream(stream, workspace)),
           "l2kv_selftest_wait_timeout")


def decode_attention_static_status(reset=False, stream=None):
    """Status word of the built-in scratch of decode_attention_static; reset=True clears it."""
    out = ctypes.c_int32(0)
    _check(lib().l2kv_decode_attention_static_status(_stream(stream), ctypes.byref(out), int(bool(reset))),
           "l2kv_decode_attention_static_status")
    return out.value


def key_norms(K, len_dev, max_len, sumsq_out, norm_out=None, stream=None, rows=None):
    lay = Layout(K, rows=rows)
    _check(lib().l2kv_key_norms(_ptr(K), lay.ref(), _ptr(len_dev), int(max_len), _ptr(sumsq_out),
                                _ptr(norm_out), _stream(stream, K)), "l2kv_key_norms")


def select_compact(K, V, len_dev, keep_dev, max_len, uncompressed_layers, K_out, V_out, idx_out,
                   sumsq_out, kept_len_dev, workspace, policy=KEEP_LOWEST_NORM, seed=0,
                   sumsq_in=None, stream=None, rows_in=None, rows_out=None):
    """rows_in / rows_out (Rows): the input / output cache is packed [Hkv, total_rows, D]."""
    lin, lout = Layout(K, rows=rows_in), Layout(K_out, rows=rows_out)
    arr, n = _layers(uncompressed_layers)
    _check(lib().l2kv_select_compact(
        _ptr(K), _ptr(V), lin.ref(), _ptr(len_dev), _ptr(keep_dev), int(max_len), arr, n,
        int(policy), ctypes.c_uint64(int(seed) & 0xFFFFFFFFFFFFFFFF), _ptr(sumsq_in), _ptr(K_out),
        _ptr(V_out), lout.ref(), _ptr(idx_out), _ptr(sumsq_out),
        _ptr(kept_len_dev), _ptr(workspace), workspace.numel(), _stream(stream, K)),
        "l2kv_select_compact")


def select_compact_per_head(K, V, len_dev, keep_unit_dev, max_len, uncompressed_layers, K_out,
                            V_out, idx_out, sumsq_out, kept_len_unit_dev, workspace,
                            policy=KEEP_LOWEST_NORM, seed=0, sumsq_in=None, stream=None):
    """select_compact with a keep count and a result length per (b, l, h)."""
    lin, lout = Layout(K), Layout(K_out)
    arr, n = _layers(uncompressed_layers)
    _check(lib().l2kv_select_compact_per_head(
        _ptr(K), _ptr(V), lin.ref(), _ptr(len_dev), _ptr(keep_unit_dev), int(max_len), arr, n,
        int(policy), ctypes.c_uint64(int(seed) & 0xFFFFFFFFFFFFFFFF), _ptr(sumsq_in), _ptr(K_out),
        _ptr(V_out), lout.ref(), _ptr(idx_out), _ptr(sumsq_out),
        _ptr(kept_len_unit_dev), _ptr(workspace), workspace.numel(), _stream(stream, K)),
        "l2kv_select_compact_per_head")


def decode_attention_per_head(q, K_c, V_c, cur_len_unit_dev, max_len, out, workspace, scale=0.0,
                              stream=None):
    """decode_attention with a cache length per (b, l, kv head)."""
    lay = Layout(K_c, q_heads=q.shape[2])
    _check(lib().l2kv_decode_attention_per_head(
        _ptr(q), _ptr(K_c), _ptr(V_c), lay.ref(), _ptr(cur_len_unit_dev), int(max_len),
        float(scale), _ptr(out), _ptr(workspace), workspace.numel(), _stream(stream, q)),
        "l2kv_decode_attention_per_head")


def decode_attention(q, K_c, V_c, cur_len_dev, max_len, out, workspace, scale=0.0, stream=None,
                     rows=None):
    lay = Layout(K_c, q_heads=q.shape[2], rows=rows)
    _check(lib().l2kv_decode_attention(
        _ptr(q), _ptr(K_c), _ptr(V_c), lay.ref(), _ptr(cur_len_dev), int(max_len), float(scale),
        _ptr(out), _ptr(workspace), workspace.numel(), _stream(stream, q)), "l2kv_decode_attention")


def append_evict(K_c, V_c, idx, sumsq_c, cur_len_dev, budget_dev, uncompressed_layers, k_new, v_new,
                 pos_new_dev, workspace, stream=None, rows=None):
    lay = Layout(K_c, rows=rows)
    arr, n = _layers(uncompressed_layers)
    _check(lib().l2kv_append_evict(
        _ptr(K_c), _ptr(V_c), _ptr(idx), _ptr(sumsq_c), lay.ref(), _ptr(cur_len_dev),
        _ptr(budget_dev), arr, n, _ptr(k_new), _ptr(v_new), _ptr(pos_new_dev), _ptr(workspace),
        workspace.numel(), _stream(stream, K_c)), "l2kv_append_evict")


def append_evict_per_head(K_c, V_c, idx, sumsq_c, cur_len_unit_dev, budget_unit_dev,
                          uncompressed_layers, k_new, v_new, pos_new_dev, workspace, stream=None):
    """append_evict with a length (in/out) and a budget per (b, l, h)."""
    lay = Layout(K_c)
    arr, n = _layers(uncompressed_layers)
    _check(lib().l2kv_append_evict_per_head(
        _ptr(K_c), _ptr(V_c), _ptr(idx), _ptr(sumsq_c), lay.ref(), _ptr(cur_len_unit_dev),
        _ptr(budget_unit_dev), arr, n, _ptr(k_new), _ptr(v_new), _ptr(pos_new_dev),
        _ptr(workspace), workspace.numel(), _stream(stream, K_c)), "l2kv_append_evict_per_head")


def decode_attention_static(q, K_c, V_c, cur_len_dev, max_len, out, scale=0.0, stream=None,
                            rows=None):
    """decode_attention for callers that cannot allocate: no workspace argument.  The partial
    results go to a fixed 16 MiB array inside the library (problems that need more raise
    L2KVError with status -4).  Calls share that array, so do not let two of them overlap on
    the GPU; make the first call on a device outside any stream capture."""
    fn = lib().l2kv_decode_attention_static
    vp = ctypes.c_void_p
    fn.restype = ctypes.c_int
    fn.argtypes = [vp, vp, vp, ctypes.POINTER(_CLayout), vp, ctypes.c_int32, ctypes.c_float, vp, vp]
    lay = Layout(K_c, q_heads=q.shape[2], rows=rows)
    _check(fn(_ptr(q), _ptr(K_c), _ptr(V_c), lay.ref(), _ptr(cur_len_dev), int(max_len),
              float(scale), _ptr(out), _stream(stream, q)), "l2kv_decode_attention_static")


def attention_loss(q, K, cur_len_dev, max_len, sumsq, alr_out, loss_out=None, loss_ref_out=None,
                   scale=0.0, workspace=None, stream=None, rows=None, per_head=False):
    """Attention loss of norm-based vs ideal compression (Eqs. 5-7); see l2kv_attention_loss.
    Allocates the (large) scratch itself unless a workspace tensor is passed.  rows (Rows): the
    cache is packed; per_head: cur_len_dev holds a length per (b, l, kv head)."""
    lay = Layout(K, q_heads=q.shape[2], rows=rows)
    if workspace is None:
        need = ctypes.c_size_t(0)
        _check(lib().l2kv_attention_loss_workspace_bytes(lay.ref(), int(max_len),
                                                         ctypes.byref(need)),
               "l2kv_attention_loss_workspace_bytes")
        workspace = torch.empty(need.value, dtype=torch.uint8, device=K.device)
    fn = lib().l2kv_attention_loss_per_head if per_head else lib().l2kv_attention_loss
    _check(fn(
        _ptr(q), _ptr(K), lay.ref(), _ptr(cur_len_dev), int(max_len), float(scale), _ptr(sumsq),
        _ptr(alr_out), _ptr(loss_out), _ptr(loss_ref_out), _ptr(workspace), workspace.numel(),
        _stream(stream, q)), "l2kv_attention_loss")


def prefix_attention_workspace(K_c, q, max_len, device=None, rows=None):
    """A zeroed workspace large enough for prefix_attention to split the cache into chunks."""
    lay = Layout(K_c, q_heads=q.shape[3], rows=rows)
    need = ctypes.c_size_t(0)
    _check(lib().l2kv_prefix_attention_workspace_bytes(lay.ref(), int(max_len), int(q.shape[2]),
                                                       ctypes.byref(need)),
           "l2kv_prefix_attention_workspace_bytes")
    return torch.zeros(need.value, dtype=torch.uint8, device=device or K_c.device)


PREFIX_CAUSAL, PREFIX_LEN_PER_HEAD, PREFIX_SPLIT_WEIGHTS = 1, 2, 4


def prefix_attention_flags(q, K_c, V_c, cur_len_dev, max_len, out, flags, lse_out=None, scale=0.0,
                           workspace=None, stream=None, rows=None):
    """The general prefix-attention call: flags is a combination of PREFIX_CAUSAL,
    PREFIX_LEN_PER_HEAD and PREFIX_SPLIT_WEIGHTS (weights as two bf16 terms: the accuracy of
    decode attention for a second P.V contraction).  rows (Rows): the cache is packed."""
    lay = Layout(K_c, q_heads=q.shape[3], rows=rows)
    _check(lib().l2kv_prefix_attention_flags(
        _ptr(q), _ptr(K_c), _ptr(V_c), lay.ref(), _ptr(cur_len_dev), int(max_len), int(q.shape[2]),
        float(scale), int(flags), _ptr(out), _ptr(lse_out), _ptr(workspace),
        0 if workspace is None else workspace.numel(), _stream(stream, q)),
        "l2kv_prefix_attention_flags")


def prefix_attention(q, K_c, V_c, cur_len_dev, max_len, out, lse_out=None, scale=0.0, workspace=None,
                     stream=None):
    """n_queries new queries per (b, l) over the compressed cache; q [B, L, Sq, Hq, D] bf16."""
    lay = Layout(K_c, q_heads=q.shape[3])
    _check(lib().l2kv_prefix_attention(
        _ptr(q), _ptr(K_c), _ptr(V_c), lay.ref(), _ptr(cur_len_dev), int(max_len), int(q.shape[2]),
        float(scale), _ptr(out), _ptr(lse_out), _ptr(workspace),
        0 if workspace is None else workspace.numel(), _stream(stream, q)), "l2kv_prefix_attention")


def prefix_attention_causal(q, K_c, V_c, cur_len_dev, max_len, out, lse_out=None, scale=0.0,
                            workspace=None, stream=None):
    """prefix_attention for a chunk whose own K/V are the last q.shape[2] cached rows: query s
    sees the rows before the chunk and the chunk up to itself."""
    lay = Layout(K_c, q_heads=q.shape[3])
    _check(lib().l2kv_prefix_attention_causal(
        _ptr(q), _ptr(K_c), _ptr(V_c), lay.ref(), _ptr(cur_len_dev), int(max_len), int(q.shape[2]),
        float(scale), _ptr(out), _ptr(lse_out), _ptr(workspace),
        0 if workspace is None else workspace.numel(), _stream(stream, q)),
        "l2kv_prefix_attention_causal")


def prefix_attention_per_head(q, K_c, V_c, cur_len_unit_dev, max_len, out, lse_out=None, scale=0.0,
                              workspace=None, stream=None):
    """prefix_attention with a cache length per (b, l, kv head)."""
    lay = Layout(K_c, q_heads=q.shape[3])
    _check(lib().l2kv_prefix_attention_per_head(
        _ptr(q), _ptr(K_c), _ptr(V_c), lay.ref(), _ptr(cur_len_unit_dev), int(max_len),
        int(q.shape[2]), float(scale), _ptr(out), _ptr(lse_out), _ptr(workspace),
        0 if workspace is None else workspace.numel(), _stream(stream, q)),
        "l2kv_prefix_attention_per_head")
