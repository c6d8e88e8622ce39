"""ctypes binding of libfact: argument marshalling only.

Every step of the computation runs in the CUDA library; PyTorch is used for
device memory (tensors, the split-K workspace) and for the current stream.
There is no fallback: if ``libfact.so`` has not been built, or the device is
not sm_100, the calls raise.

The raw C entry points are available under their C names on ``lib()``
(``lib().fact_gemm`` ...); ``Handle`` wraps them for torch tensors.
"""
from __future__ import annotations

import ctypes
from ctypes import POINTER, Structure, byref, c_char_p, c_double, c_float, c_int, c_int64, c_size_t, c_void_p
from pathlib import Path
from typing import Optional

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libfact.so"

OK = 0
STATUS_NAMES = {
    0: "FACT_OK", 1: "FACT_ERR_INVALID_ARG", 2: "FACT_ERR_BAD_ALIGNMENT", 3: "FACT_ERR_UNSUPPORTED",
    4: "FACT_ERR_ARCH", 5: "FACT_ERR_WORKSPACE_TOO_SMALL", 6: "FACT_ERR_CUDA", 7: "FACT_ERR_DEVICE_TIMEOUT",
}
EPILOGUES = {"NONE": 0, "BIAS": 1, "BIAS_RELU": 2, "BIAS_GELU_TANH": 3, "SILU_GATE": 4, "BIAS_RESIDUAL": 5,
             "BIAS_SOFTMAX": 6}
LAYOUTS = {"KN": 0, "NK": 1}
OUT_TYPES = {torch.bfloat16: 0, torch.float32: 1, "bf16": 0, "f32": 1}
OPS = {"gemm": 0, "gemm_batched": 1, "gemm_splitk": 2, "linear": 3, "linear_fp8": 4}

# every symbol include/fact.h declares
EXPORTED = [
    "fact_create", "fact_destroy", "fact_status_string", "fact_workspace_bytes", "fact_gemm", "fact_gemm_batched",
    "fact_gemm_splitk", "fact_linear", "fact_get_config", "fact_tune", "fact_tune_cache_save",
    "fact_tune_cache_load", "fact_device_status", "fact_launch_count", "fact_device_info", "fact_last_error",
    "fact_last_kernel_clock", "fact_gemm_splitk_static", "fact_last_kernel_profile", "fact_selftest_wait_timeout",
    "fact_attention", "fact_norm", "fact_block_workspace_bytes", "fact_block_workspace_offsets", "fact_block_forward",
    "fact_stream_k_pieces", "fact_attention_deal", "fact_linear_fp8", "fact_linear_grouped", "fact_linear_grouped_fp8",
    "fact_linear_ex", "fact_row_stats", "fact_fold_norm", "fact_gemm_splitk_static_status", "fact_debug_flags",
    "fact_tune_ex", "fact_last_kernel_span", "fact_gemm_host", "fact_gemm_host_scratch_bytes",
    "fact_gemm_host_wait",
]


NORMS = {"layer": 0, "rms": 1}
XNORMS = {None: 0, "none": 0, "layer": 1, "rms": 2}


class LinearExt(Structure):
    """Mirror of fact_linear_ext_t."""

    _fields_ = [("row_stats_out", c_void_p), ("x_norm", c_int), ("x_row_stats", c_void_p), ("w_colsum", c_void_p),
                ("eps", c_float)]
BLOCK_KINDS = {"gpt": 0, "llama": 1}


class Block(Structure):
    """Mirror of fact_block_t."""

    _fields_ = ([("kind", c_int)] +
                [(n, c_int64) for n in ("batch", "seq", "hidden", "heads_q", "heads_kv", "head_dim", "ffn")] +
                [("eps", c_float)] +
                [(n, c_void_p) for n in ("norm1_gamma", "norm1_beta", "wqkv", "bqkv", "wo", "bo", "norm2_gamma",
                                         "norm2_beta", "w1", "b1", "w2", "b2")])


TUNE_OUTCOMES = {0: "timed", 1: "infeasible", 2: "no_workspace", 3: "launch_failed", 4: "verify_failed"}


class FactError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {STATUS_NAMES.get(code, code)}")


class Config(Structure):
    """Mirror of fact_config_t; zero fields mean "library's choice"."""

    _fields_ = [(n, c_int) for n in
                ("tile_m", "tile_n", "tile_k", "stages", "cta_group", "raster_group", "split_k", "store_mode", "schedule")]

    def as_dict(self):
        return {n: int(getattr(self, n)) for n, _ in self._fields_}

    def __repr__(self):
        return "Config(" + ", ".join(f"{k}={v}" for k, v in self.as_dict().items()) + ")"


class TuneRecord(Structure):
    """Mirror of fact_tune_record_t: what the tuner did with one candidate."""

    _fields_ = [("cfg", Config), ("status", c_int), ("ms", c_float), ("rel", c_float), ("verify_err", c_float)]

    def as_dict(self):
        return {"cfg": self.cfg.as_dict(), "outcome": TUNE_OUTCOMES.get(int(self.status), int(self.status)),
                "ms": float(self.ms), "rel": float(self.rel), "verify_err": float(self.verify_err)}


class TuneOpts(Structure):
    """Mirror of fact_tune_opts_t."""

    _fields_ = [("cold_l2", c_int), ("verify", c_int), ("inject_fault", c_int), ("records", POINTER(TuneRecord)),
                ("max_records", c_int), ("n_records", POINTER(c_int))]


_lib = None


def lib() -> ctypes.CDLL:
    """Load libfact.so (built in-tree by ``python -m paper_2604_26666_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not LIB_PATH.exists():
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2604_26666_b200.build` "
                           "(there is no fallback path)")
    L = ctypes.CDLL(str(LIB_PATH))
    i64, vp, sz = c_int64, c_void_p, c_size_t
    cfgp = POINTER(Config)
    L.fact_create.argtypes = [POINTER(vp), c_int]
    L.fact_destroy.argtypes = [vp]
    L.fact_status_string.argtypes = [c_int]
    L.fact_status_string.restype = c_char_p
    L.fact_workspace_bytes.argtypes = [vp, c_int, i64, i64, i64, i64, c_int, c_int, c_int, cfgp, POINTER(sz)]
    L.fact_gemm.argtypes = [vp, i64, i64, i64, vp, i64, vp, i64, c_int, vp, i64, c_int, cfgp, vp, sz, vp]
    L.fact_gemm_batched.argtypes = [vp, i64, i64, i64, i64, vp, i64, i64, vp, i64, i64, c_int, vp, i64, i64, c_int,
                                    cfgp, vp, sz, vp]
    L.fact_gemm_splitk.argtypes = [vp, i64, i64, i64, vp, i64, vp, i64, c_int, vp, i64, c_int, c_int, cfgp, vp, sz, vp]
    L.fact_gemm_splitk_static.argtypes = [c_int, i64, i64, i64, vp, i64, vp, i64, c_int, vp, i64, c_int, c_int, vp]
    L.fact_attention.argtypes = [vp, i64, i64, i64, i64, i64, i64, vp, i64, i64, i64, vp, i64, i64, i64, vp, i64, i64, i64,
                                 vp, i64, i64, i64, c_int, ctypes.c_float, vp]
    L.fact_linear.argtypes = [vp, i64, i64, i64, vp, i64, vp, i64, c_int, vp, vp, i64, vp, i64, c_int, c_int, cfgp,
                              vp, sz, vp]
    L.fact_get_config.argtypes = [vp, c_int, i64, i64, i64, i64, c_int, c_int, c_int, cfgp]
    L.fact_tune.argtypes = [vp, c_int, i64, i64, i64, i64, vp, i64, i64, vp, i64, i64, c_int, vp, vp, i64, i64, vp,
                            i64, i64, c_int, c_int, vp, sz, c_int, c_int, vp, cfgp, POINTER(c_double), POINTER(c_int)]
    L.fact_tune_ex.argtypes = [vp, c_int, i64, i64, i64, i64, vp, i64, i64, vp, i64, i64, c_int, vp, vp, i64, i64, vp,
                               i64, i64, c_int, c_int, vp, sz, c_int, c_int, vp, POINTER(TuneOpts), cfgp,
                               POINTER(c_double), POINTER(c_int)]
    L.fact_tune_cache_save.argtypes = [vp, c_char_p]
    L.fact_tune_cache_load.argtypes = [vp, c_char_p]
    L.fact_device_status.argtypes = [vp, vp, POINTER(c_int)]
    L.fact_launch_count.argtypes = [vp]
    L.fact_launch_count.restype = i64
    L.fact_device_info.argtypes = [vp, POINTER(c_int), POINTER(c_int), POINTER(c_int), POINTER(c_int)]
    L.fact_last_kernel_clock.argtypes = [vp, vp, POINTER(i64), POINTER(i64)]
    L.fact_last_kernel_profile.argtypes = [vp, vp, POINTER(i64)]
    L.fact_selftest_wait_timeout.argtypes = [vp, vp, c_double]
    L.fact_last_error.argtypes = [vp]
    L.fact_last_error.restype = c_char_p
    L.fact_norm.argtypes = [vp, c_int, i64, i64, vp, i64, vp, vp, c_float, vp, i64, vp]
    L.fact_block_workspace_bytes.argtypes = [POINTER(Block)]
    L.fact_block_workspace_bytes.restype = sz
    L.fact_block_workspace_offsets.argtypes = [POINTER(Block), POINTER(sz)]
    L.fact_block_forward.argtypes = [vp, POINTER(Block), vp, vp, vp, sz, vp]
    L.fact_linear_fp8.argtypes = [vp, i64, i64, i64, vp, i64, vp, i64, c_float, vp, vp, i64, vp, i64, c_int, c_int, cfgp,
                                  vp, sz, vp]
    L.fact_linear_grouped.argtypes = [vp, c_int, POINTER(i64), i64, i64, vp, i64, vp, i64, i64, c_int, vp, vp, i64, vp, i64,
                                      c_int, c_int, cfgp, vp]
    L.fact_linear_grouped_fp8.argtypes = [vp, c_int, POINTER(i64), i64, i64, vp, i64, vp, i64, i64, c_float, vp, vp, i64, vp,
                                          i64, c_int, c_int, cfgp, vp]
    L.fact_linear_ex.argtypes = [vp, i64, i64, i64, vp, i64, vp, i64, c_int, vp, vp, i64, vp, i64, c_int, c_int,
                                 POINTER(LinearExt), cfgp, vp, sz, vp]
    L.fact_row_stats.argtypes = [vp, i64, i64, vp, i64, vp, vp]
    L.fact_fold_norm.argtypes = [vp, i64, i64, vp, i64, vp, vp, vp, vp, i64, vp, vp, vp]
    L.fact_stream_k_pieces.argtypes = [c_int, i64, i64, c_int, c_int, POINTER(ctypes.c_int32), POINTER(c_int)]
    L.fact_attention_deal.argtypes = [c_int, i64, i64, c_int, c_int, c_int, POINTER(ctypes.c_int32), POINTER(c_int)]
    L.fact_gemm_splitk_static_status.argtypes = [c_int, vp, POINTER(c_int)]
    L.fact_debug_flags.argtypes = [vp]
    L.fact_last_kernel_span.argtypes = [vp, vp, POINTER(i64)]
    L.fact_gemm_host_scratch_bytes.argtypes = [vp, i64, i64, i64, c_int, c_int, cfgp, POINTER(sz)]
    L.fact_gemm_host_wait.argtypes = [vp, vp]
    L.fact_gemm_host.argtypes = [vp, i64, i64, i64, vp, i64, vp, i64, c_int, vp, i64, c_int, cfgp, vp, sz, vp]
    for name in EXPORTED:
        fn = getattr(L, name)
        if name not in ("fact_status_string", "fact_launch_count", "fact_last_error", "fact_block_workspace_bytes"):
            fn.restype = c_int
    _lib = L
    return L


def _check(code: int, where: str, handle=None):
    if code != OK:
        if code == 6 and handle is not None:
            where += " [" + (lib().fact_last_error(handle) or b"").decode() + "]"
        raise FactError(code, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else c_void_p(t.data_ptr())


def _need(t: torch.Tensor, name: str, dtype, ndim, cuda: bool = True):
    if not isinstance(t, torch.Tensor):
        raise TypeError(f"{name} must be a tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if t.ndim != ndim:
        raise ValueError(f"{name} must have {ndim} dimensions")
    if t.shape[-1] > 1 and t.stride(-1) != 1:
        raise ValueError(f"{name}: innermost dimension must be contiguous")
    if cuda and not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")


def _need_out(out: torch.Tensor, shape, like: torch.Tensor, name: str = "out"):
    """A caller-supplied output must have exactly the result's shape, a supported dtype, and live on the operands'
    device: the kernels write `shape` elements through its pointer whatever its real size is."""
    if not isinstance(out, torch.Tensor):
        raise TypeError(f"{name} must be a tensor")
    if out.dtype not in (torch.bfloat16, torch.float32):
        raise TypeError(f"{name} must be bfloat16 or float32, got {out.dtype}")
    if tuple(out.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(out.shape)}")
    if out.device != like.device:
        raise ValueError(f"{name} is on {out.device}, the operands are on {like.device}")
    if out.shape[-1] > 1 and out.stride(-1) != 1:
        raise ValueError(f"{name}: innermost dimension must be contiguous")
    if not out.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")


def _validate_matmul(A, B, out, layout: str, batched: bool = False):
    """Shape, dtype and device checks of C = A @ B before anything is handed to the library (a mismatch there would
    be an out-of-bounds device access, not an error code).  Shape errors are reported before the tensors are required
    to be on a GPU.  Returns (batch, M, N, K)."""
    nd = 3 if batched else 2
    _need(A, "A", torch.bfloat16, nd, cuda=False)
    _need(B, "B", torch.bfloat16, nd, cuda=False)
    if layout not in LAYOUTS:
        raise ValueError(f"layout must be one of {sorted(LAYOUTS)}")
    M, K = A.shape[-2:]
    N, Kb = (B.shape[-1], B.shape[-2]) if layout == "KN" else (B.shape[-2], B.shape[-1])
    if Kb != K:
        raise ValueError(f"inner dimensions differ: A has K = {K}, B has K = {Kb}")
    batch = A.shape[0] if batched else 1
    if batched and B.shape[0] != batch:
        raise ValueError("batch sizes differ")
    _same_device(A, B)
    if out is not None:
        _need_out(out, (batch, M, N) if batched else (M, N), A)
    for name, t in (("A", A), ("B", B)):
        if not t.is_cuda:
            raise TypeError(f"{name} must be a CUDA tensor")
    return int(batch), int(M), int(N), int(K)


def _same_device(*tensors):
    devs = {t.device for t in tensors if t is not None}
    if len(devs) > 1:
        raise ValueError(f"tensors live on different devices: {sorted(str(d) for d in devs)}")


def _ld(t: torch.Tensor) -> int:
    """Leading dimension of the last two dims; a one-row matrix may carry any stride."""
    return int(t.stride(-2)) if t.shape[-2] > 1 else max(int(t.shape[-1]), int(t.stride(-2)))


def stream_k_pieces(groups: int, sk_tiles: int, k_blocks: int, group: int):
    """The stream-K pieces of one CTA group (fact_stream_k_pieces; host arithmetic, no device needed):
    a list of (tile, k_begin, k_end, role, peers)."""
    cap = 8
    while True:
        buf = (ctypes.c_int32 * (5 * cap))()
        n = c_int(0)
        _check(lib().fact_stream_k_pieces(groups, sk_tiles, k_blocks, group, cap, buf, byref(n)),
               "fact_stream_k_pieces")
        if n.value <= cap:
            return [tuple(buf[5 * i: 5 * i + 5]) for i in range(n.value)]
        cap = n.value


def attention_deal(ctas: int, batch_heads: int, seq: int, head_dim: int, cta: int):
    """The items one CTA of a causal attention call takes (fact_attention_deal; host arithmetic, no device needed)."""
    cap = 64
    while True:
        buf = (ctypes.c_int32 * cap)()
        n = c_int(0)
        _check(lib().fact_attention_deal(ctas, batch_heads, seq, head_dim, cta, cap, buf, byref(n)), "fact_attention_deal")
        if n.value <= cap:
            return list(buf[: n.value])
        cap = n.value


def gemm_splitk_static(A, B, out, layout="KN", splits=0, device=None, stream=None):
    """C = A @ B through fact_gemm_splitk_static: no handle, no workspace, no device allocation inside the
    library (its split-K scratch is a fixed 16 MiB array inside the library image).  For callers that may
    not call cudaMalloc; `out` must be preallocated by the caller.  Calls on one device must not overlap."""
    if out is None:
        raise TypeError("out must be preallocated by the caller: this entry point exists for callers that cannot allocate")
    _, M, N, K = _validate_matmul(A, B, out, layout)
    dev = A.device.index if device is None else int(device)
    if dev != A.device.index:
        raise ValueError(f"the operands are on cuda:{A.device.index}, the call names device {dev}")
    s = stream if stream is not None else torch.cuda.current_stream(dev)
    _check(lib().fact_gemm_splitk_static(dev, M, N, K, _ptr(A), _ld(A), _ptr(B), _ld(B), LAYOUTS[layout], _ptr(out),
                                         _ld(out), OUT_TYPES[out.dtype], int(splits), c_void_p(s.cuda_stream)),
           "fact_gemm_splitk_static")
    return out


def gemm_splitk_static_status(device: int = 0, stream=None) -> int:
    """The device status word of fact_gemm_splitk_static on `device` (0, or 7 after a device-side wait gave up:
    the output of that call is then undefined); synchronises the stream and clears the word."""
    s = stream if stream is not None else torch.cuda.current_stream(device)
    v = c_int(0)
    _check(lib().fact_gemm_splitk_static_status(int(device), c_void_p(s.cuda_stream), byref(v)),
           "fact_gemm_splitk_static_status")
    return int(v.value)


class Handle:
    """A libfact handle on one CUDA device, plus a grow-only torch workspace."""

    def __init__(self, device: int = 0, load_table: bool = True):
        self._h = c_void_p()
        self.device = int(device)
        _check(lib().fact_create(byref(self._h), self.device), "fact_create")
        self._ws: Optional[torch.Tensor] = None
        self._ws_streams: dict = {}
        self._ws_cache: dict = {}
        table = _PKG / "tuned_b200.txt"
        if load_table and table.exists():  # the tuner's table for the benchmark shapes, measured on a B200
            self.tune_cache_load(str(table))

    def close(self):
        if self._h:
            lib().fact_destroy(self._h)
            self._h = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- helpers ------------------------------------------------------------------------------
    def _stream(self, stream) -> c_void_p:
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        self._ws_streams[int(s.cuda_stream)] = s  # kernels on this stream may be using the workspace
        return c_void_p(s.cuda_stream)

    def _cfg(self, cfg):
        if cfg is None:
            return None
        if isinstance(cfg, Config):
            return byref(cfg)
        c = Config(**{k: int(v) for k, v in dict(cfg).items()})
        return byref(c)

    def workspace(self, nbytes: int) -> Optional[torch.Tensor]:
        if nbytes <= 0:
            return None
        if self._ws is None or self._ws.numel() < nbytes:
            if self._ws is not None:
                # kernels launched on other streams than torch's current one may still read the old buffer: tell the
                # caching allocator, so that it does not hand the block out again before they have finished
                for s in self._ws_streams.values():
                    self._ws.record_stream(s)
            self._ws = torch.empty(nbytes, dtype=torch.uint8, device=f"cuda:{self.device}")
        return self._ws

    def workspace_bytes(self, op, batch, M, N, K, epilogue="NONE", layout="KN", out_dtype=torch.bfloat16, cfg=None,
                        splits=0) -> int:
        if cfg is None or isinstance(cfg, Config):
            ckey = None if cfg is None else tuple(cfg.as_dict().values())
        else:
            ckey = tuple(sorted(dict(cfg).items()))
        key = (op, batch, M, N, K, epilogue, layout, out_dtype, ckey, splits)
        hit = self._ws_cache.get(key)
        if hit is not None:
            return hit
        n = c_size_t(0)
        c = self._cfg_with_splits(cfg, splits)
        _check(lib().fact_workspace_bytes(self._h, OPS[op], batch, M, N, K, EPILOGUES[epilogue], LAYOUTS[layout],
                                          OUT_TYPES[out_dtype], c, byref(n)), "fact_workspace_bytes")
        self._ws_cache[key] = int(n.value)
        return int(n.value)

    def _cfg_with_splits(self, cfg, splits):
        if not splits:
            return self._cfg(cfg)
        d = cfg.as_dict() if isinstance(cfg, Config) else dict(cfg or {})
        d["split_k"] = int(splits)
        return self._cfg(d)

    def get_config(self, op, batch, M, N, K, epilogue="NONE", layout="KN", out_dtype=torch.bfloat16) -> Config:
        c = Config()
        _check(lib().fact_get_config(self._h, OPS[op], batch, M, N, K, EPILOGUES[epilogue], LAYOUTS[layout],
                                     OUT_TYPES[out_dtype], byref(c)), "fact_get_config")
        return c

    def device_status(self, stream=None) -> int:
        v = c_int(0)
        _check(lib().fact_device_status(self._h, self._stream(stream), byref(v)), "fact_device_status")
        return int(v.value)

    def last_kernel_clock(self, stream=None):
        """(SM cycles, nanoseconds) of the first CTA of the last GEMM launch; their ratio is the SM clock in GHz."""
        c, n = c_int64(0), c_int64(0)
        _check(lib().fact_last_kernel_clock(self._h, self._stream(stream), byref(c), byref(n)), "fact_last_kernel_clock")
        return int(c.value), int(n.value)

    def last_kernel_profile(self, stream=None):
        """The eight cycle counters of fact_last_kernel_profile (needs FACT_DEBUG_FLAGS=256)."""
        arr = (c_int64 * 8)()
        _check(lib().fact_last_kernel_profile(self._h, self._stream(stream), arr), "fact_last_kernel_profile")
        return [int(x) for x in arr]

    def last_kernel_span(self, stream=None) -> int:
        """Nanoseconds from the first CTA's start to the last CTA's end of the last GEMM launch (FACT_DEBUG_FLAGS=256)."""
        v = c_int64(0)
        _check(lib().fact_last_kernel_span(self._h, self._stream(stream), byref(v)), "fact_last_kernel_span")
        return int(v.value)

    def selftest_wait_timeout(self, limit_ms: float = 5.0, stream=None):
        """Run the bounded-wait self-test (fact_selftest_wait_timeout); raises unless the wait gave up cleanly."""
        _check(lib().fact_selftest_wait_timeout(self._h, self._stream(stream), float(limit_ms)),
               "fact_selftest_wait_timeout", self._h)

    def debug_flags(self) -> int:
        """The FACT_DEBUG_FLAGS bits in effect (0 in normal use; the default build honours diagnostics only)."""
        return int(lib().fact_debug_flags(self._h))

    def launch_count(self) -> int:
        return int(lib().fact_launch_count(self._h))

    def device_info(self) -> dict:
        a, b, c, d = c_int(), c_int(), c_int(), c_int()
        _check(lib().fact_device_info(self._h, byref(a), byref(b), byref(c), byref(d)), "fact_device_info")
        return {"sm_count": a.value, "max_smem_per_block": b.value, "cc": (c.value, d.value)}

    def tune_cache_save(self, path: str):
        _check(lib().fact_tune_cache_save(self._h, str(path).encode()), "fact_tune_cache_save")

    def tune_cache_load(self, path: str):
        _check(lib().fact_tune_cache_load(self._h, str(path).encode()), "fact_tune_cache_load")
        self._ws_cache.clear()  # the library's own choices may have changed

    # -- compute ------------------------------------------------------------------------------
    def gemm(self, A, B, layout="KN", out=None, out_dtype=torch.bfloat16, cfg=None, stream=None):
        """C = A @ B  (fact_gemm).  layout "KN": B is [K, N]; "NK": B is [N, K]."""
        _, M, N, K = _validate_matmul(A, B, out, layout)
        if out is None:
            out = torch.empty((M, N), dtype=out_dtype, device=A.device)
        c = self._cfg(cfg)
        nws = self.workspace_bytes("gemm", 1, M, N, K, "NONE", layout, out.dtype, cfg)
        ws = self.workspace(nws)
        _check(lib().fact_gemm(self._h, M, N, K, _ptr(A), _ld(A), _ptr(B), _ld(B), LAYOUTS[layout], _ptr(out),
                               _ld(out), OUT_TYPES[out.dtype], c, _ptr(ws), nws, self._stream(stream)), "fact_gemm", self._h)
        return out

    def gemm_host(self, A, B, out, scratch, layout="KN", cfg=None, stream=None):
        """C = A @ B for HOST tensors (fact_gemm_host): A, B BF16 CPU tensors (pinned for asynchronous copies), `out`
        a BF16 or FP32 CPU tensor, `scratch` a device uint8 tensor of at least gemm_host_scratch_bytes(...) bytes.
        Enqueues copy-in, product and copy-out on the handle's own three streams; `out` is valid after
        gemm_host_wait() and a synchronisation of that stream.  Give consecutive calls different scratch tensors and
        their copies overlap each other's products."""
        nd = 2
        _need(A, "A", torch.bfloat16, nd, cuda=False)
        _need(B, "B", torch.bfloat16, nd, cuda=False)
        if A.is_cuda or B.is_cuda or out.is_cuda:
            raise TypeError("gemm_host takes host tensors; use gemm for device tensors")
        M, K = A.shape
        N, Kb = (B.shape[1], B.shape[0]) if layout == "KN" else (B.shape[0], B.shape[1])
        if Kb != K:
            raise ValueError(f"inner dimensions differ: A has K = {K}, B has K = {Kb}")
        if out.dtype not in (torch.bfloat16, torch.float32) or tuple(out.shape) != (M, N):
            raise ValueError(f"out must be a bfloat16 or float32 host tensor of shape {(M, N)}")
        if out.shape[-1] > 1 and out.stride(-1) != 1:
            raise ValueError("out: innermost dimension must be contiguous")
        need = self.gemm_host_scratch_bytes(M, N, K, out.dtype, layout, cfg)
        if not (isinstance(scratch, torch.Tensor) and scratch.is_cuda and scratch.dtype == torch.uint8
                and scratch.is_contiguous() and scratch.numel() >= need and scratch.device.index == self.device):
            raise ValueError(f"scratch must be a contiguous uint8 tensor of at least {need} bytes on cuda:{self.device}")
        _check(lib().fact_gemm_host(self._h, M, N, K, _ptr(A), _ld(A), _ptr(B), _ld(B), LAYOUTS[layout], _ptr(out),
                                    _ld(out), OUT_TYPES[out.dtype], self._cfg(cfg), _ptr(scratch), scratch.numel(),
                                    self._stream(stream)), "fact_gemm_host", self._h)
        return out

    def gemm_host_wait(self, stream=None):
        """Make `stream` (default: torch's current stream) wait for the copy-out of every gemm_host call so far."""
        _check(lib().fact_gemm_host_wait(self._h, self._stream(stream)), "fact_gemm_host_wait", self._h)

    def gemm_host_scratch_bytes(self, M, N, K, out_dtype=torch.bfloat16, layout="KN", cfg=None) -> int:
        """Device scratch a gemm_host call of this shape needs: the operands' device copies and the product's workspace."""
        n = c_size_t(0)
        _check(lib().fact_gemm_host_scratch_bytes(self._h, M, N, K, LAYOUTS[layout], OUT_TYPES[out_dtype],
                                                  self._cfg(cfg), byref(n)), "fact_gemm_host_scratch_bytes")
        return int(n.value)

    def gemm_batched(self, A, B, layout="KN", out=None, out_dtype=torch.bfloat16, cfg=None, stream=None):
        """C[b] = A[b] @ B[b]  (fact_gemm_batched)."""
        batch, M, N, K = _validate_matmul(A, B, out, layout, batched=True)
        if out is None:
            out = torch.empty((batch, M, N), dtype=out_dtype, device=A.device)
        nws = self.workspace_bytes("gemm_batched", batch, M, N, K, "NONE", layout, out.dtype, cfg)
        ws = self.workspace(nws)
        _check(lib().fact_gemm_batched(self._h, batch, M, N, K, _ptr(A), _ld(A), A.stride(0), _ptr(B), _ld(B),
                                       B.stride(0), LAYOUTS[layout], _ptr(out), _ld(out), out.stride(0),
                                       OUT_TYPES[out.dtype], self._cfg(cfg), _ptr(ws), nws, self._stream(stream)),
               "fact_gemm_batched", self._h)
        return out

    def gemm_splitk(self, A, B, layout="KN", out=None, out_dtype=torch.float32, splits=0, cfg=None, stream=None):
        """C = A @ B with K cut into slices and a fixed-order reduction  (fact_gemm_splitk)."""
        _, M, N, K = _validate_matmul(A, B, out, layout)
        if out is None:
            out = torch.empty((M, N), dtype=out_dtype, device=A.device)
        nws = self.workspace_bytes("gemm_splitk", 1, M, N, K, "NONE", layout, out.dtype, cfg, splits)
        ws = self.workspace(nws)
        _check(lib().fact_gemm_splitk(self._h, M, N, K, _ptr(A), _ld(A), _ptr(B), _ld(B), LAYOUTS[layout], _ptr(out),
                                      _ld(out), OUT_TYPES[out.dtype], int(splits), self._cfg(cfg), _ptr(ws), nws,
                                      self._stream(stream)), "fact_gemm_splitk", self._h)
        return out

    def linear(self, X, W, bias=None, residual=None, epilogue="NONE", layout="NK", out=None,
               out_dtype=torch.bfloat16, cfg=None, stream=None, stats_out=None, x_norm=None, x_stats=None,
               w_colsum=None, eps=1e-5):
        """Y = epilogue(X @ W)  (fact_linear).  layout "NK": W is [Nw, K] (nn.Linear weight); "KN": [K, Nw].
        For SILU_GATE W carries 2*N_out columns (gate first, then up).
        stats_out (FP32 [ceil(N_out/64), M, 2]) receives partial row sums of Y; x_norm "layer" / "rms" with x_stats
        (and w_colsum for "layer") folds a normalisation of X's rows into the product (fact_linear_ex)."""
        _need(X, "X", torch.bfloat16, 2)
        _need(W, "W", torch.bfloat16, 2)
        M, K = X.shape
        Nw = W.shape[1] if layout == "KN" else W.shape[0]
        if (W.shape[0] if layout == "KN" else W.shape[1]) != K:
            raise ValueError("inner dimensions differ")
        if epilogue == "SILU_GATE":
            if Nw % 2:
                raise ValueError("SILU_GATE needs an even number of weight columns")
            N = Nw // 2
        else:
            N = Nw
        if bias is not None:
            _need(bias, "bias", torch.bfloat16, 1)
            if bias.shape[0] != N:
                raise ValueError("bias must have N_out entries")
        if residual is not None:
            _need(residual, "residual", torch.bfloat16, 2)
            if tuple(residual.shape) != (M, N):
                raise ValueError("residual must be [M, N_out]")
        _same_device(X, W, bias, residual)
        if out is None:
            out = torch.empty((M, N), dtype=out_dtype, device=X.device)
        _need_out(out, (M, N), X)
        nws = self.workspace_bytes("linear", 1, M, N, K, epilogue, layout, out.dtype, cfg)
        ws = self.workspace(nws)
        if stats_out is not None or x_norm not in (None, "none") or x_stats is not None or w_colsum is not None:
            if stats_out is not None:
                _need(stats_out, "stats_out", torch.float32, 3)
                if tuple(stats_out.shape) != ((N + 63) // 64, M, 2) or not stats_out.is_contiguous():
                    raise ValueError("stats_out must be a contiguous [ceil(N_out/64), M, 2]")
            if x_stats is not None:
                _need(x_stats, "x_stats", torch.float32, 3)
                if tuple(x_stats.shape) != ((K + 63) // 64, M, 2) or not x_stats.is_contiguous():
                    raise ValueError("x_stats must be a contiguous [ceil(K/64), M, 2]")
            if w_colsum is not None:
                _need(w_colsum, "w_colsum", torch.float32, 1)
                if w_colsum.shape[0] != N:
                    raise ValueError("w_colsum must have N_out entries")
            ext = LinearExt(_ptr(stats_out), XNORMS[x_norm], _ptr(x_stats), _ptr(w_colsum), float(eps))
            _check(lib().fact_linear_ex(self._h, M, N, K, _ptr(X), _ld(X), _ptr(W), _ld(W), LAYOUTS[layout],
                                        _ptr(bias), _ptr(residual), _ld(residual) if residual is not None else 0,
                                        _ptr(out), _ld(out), OUT_TYPES[out.dtype], EPILOGUES[epilogue],
                                        ctypes.byref(ext), self._cfg(cfg), _ptr(ws), nws, self._stream(stream)),
                   "fact_linear_ex", self._h)
            return out
        _check(lib().fact_linear(self._h, M, N, K, _ptr(X), _ld(X), _ptr(W), _ld(W), LAYOUTS[layout], _ptr(bias),
                                 _ptr(residual), _ld(residual) if residual is not None else 0, _ptr(out), _ld(out),
                                 OUT_TYPES[out.dtype], EPILOGUES[epilogue], self._cfg(cfg), _ptr(ws), nws,
                                 self._stream(stream)), "fact_linear", self._h)
        return out

    def row_stats(self, X, out=None, stream=None):
        """Partial row sums of X per 64-column chunk: FP32 [ceil(C/64), M, 2] (fact_row_stats)."""
        _need(X, "X", torch.bfloat16, 2)
        M, C = X.shape
        if out is None:
            out = torch.empty(((C + 63) // 64, M, 2), dtype=torch.float32, device=X.device)
        _need(out, "out", torch.float32, 3)
        _check(lib().fact_row_stats(self._h, M, C, _ptr(X), _ld(X), _ptr(out), self._stream(stream)),
               "fact_row_stats", self._h)
        return out

    def fold_norm(self, W, gamma, beta=None, bias=None, stream=None):
        """Fold a normalisation's gamma (and beta) into the [N_w, K] weights of the layer after it (fact_fold_norm).
        Returns (W_folded, colsum, bias_folded); bias_folded is None without beta."""
        _need(W, "W", torch.bfloat16, 2)
        _need(gamma, "gamma", torch.bfloat16, 1)
        Nw, K = W.shape
        if gamma.shape[0] != K:
            raise ValueError("gamma must have K entries")
        if beta is not None:
            _need(beta, "beta", torch.bfloat16, 1)
        if bias is not None:
            _need(bias, "bias", torch.bfloat16, 1)
        Wf = torch.empty_like(W)
        colsum = torch.empty(Nw, dtype=torch.float32, device=W.device)
        bf = torch.empty(Nw, dtype=torch.bfloat16, device=W.device) if beta is not None else None
        _check(lib().fact_fold_norm(self._h, Nw, K, _ptr(W), _ld(W), _ptr(gamma), _ptr(beta), _ptr(bias), _ptr(Wf),
                                    _ld(Wf), _ptr(colsum), _ptr(bf), self._stream(stream)), "fact_fold_norm", self._h)
        return Wf, colsum, bf

    def linear_grouped(self, X, W, group_rows, bias=None, residual=None, epilogue="NONE", layout="NK", out=None,
                       out_dtype=torch.bfloat16, cfg=None, stream=None):
        """Y[rows of group g] = epilogue(X[rows of group g] @ W[g])  (fact_linear_grouped).  X [M, K]; W [G, Nw, K]
        (layout "NK") or [G, K, Nw] ("KN"); group_rows: G row counts summing to M (host integers)."""
        _need(X, "X", torch.bfloat16, 2)
        _need(W, "W", torch.bfloat16, 3)
        rows = [int(r) for r in group_rows]
        G = len(rows)
        M, K = X.shape
        if W.shape[0] != G or sum(rows) != M:
            raise ValueError("group_rows must have one entry per weight matrix and sum to the rows of X")
        Nw = W.shape[2] if layout == "KN" else W.shape[1]
        if (W.shape[1] if layout == "KN" else W.shape[2]) != K:
            raise ValueError("inner dimensions differ")
        N = Nw // 2 if epilogue == "SILU_GATE" else Nw
        if bias is not None:
            _need(bias, "bias", torch.bfloat16, 1)
        if residual is not None:
            _need(residual, "residual", torch.bfloat16, 2)
        if out is None:
            out = torch.empty((M, N), dtype=out_dtype, device=X.device)
        _need_out(out, (M, N), X)
        arr = (c_int64 * max(G, 1))(*rows)
        _check(lib().fact_linear_grouped(self._h, G, arr, N, K, _ptr(X), _ld(X), _ptr(W), _ld(W),
                                         int(W.stride(0)) if G > 1 else int(W.shape[1] * W.stride(1)), LAYOUTS[layout],
                                         _ptr(bias), _ptr(residual), _ld(residual) if residual is not None else 0,
                                         _ptr(out), _ld(out), OUT_TYPES[out.dtype], EPILOGUES[epilogue], self._cfg(cfg),
                                         self._stream(stream)), "fact_linear_grouped", self._h)
        return out

    def linear_grouped_fp8(self, X, W, group_rows, scale=1.0, bias=None, epilogue="NONE", out=None,
                           out_dtype=torch.bfloat16, cfg=None, stream=None):
        """fact_linear_grouped_fp8: X [M, K] and W [G, Nw, K] are FP8 E4M3 (torch.float8_e4m3fn or uint8 codes)."""
        def codes(t, name, nd):
            if isinstance(t, torch.Tensor) and t.dtype == torch.float8_e4m3fn:
                t = t.view(torch.uint8)
            _need(t, name, torch.uint8, nd)
            return t
        X, W = codes(X, "X", 2), codes(W, "W", 3)
        rows = [int(r) for r in group_rows]
        G = len(rows)
        M, K = X.shape
        if W.shape[0] != G or sum(rows) != M or W.shape[2] != K:
            raise ValueError("shapes differ")
        Nw = W.shape[1]
        N = Nw // 2 if epilogue == "SILU_GATE" else Nw
        if bias is not None:
            _need(bias, "bias", torch.bfloat16, 1)
        if out is None:
            out = torch.empty((M, N), dtype=out_dtype, device=X.device)
        _need_out(out, (M, N), X)
        arr = (c_int64 * max(G, 1))(*rows)
        _check(lib().fact_linear_grouped_fp8(self._h, G, arr, N, K, _ptr(X), _ld(X), _ptr(W), _ld(W),
                                             int(W.stride(0)) if G > 1 else int(W.shape[1] * W.stride(1)), float(scale),
                                             _ptr(bias), None, 0, _ptr(out), _ld(out), OUT_TYPES[out.dtype],
                                             EPILOGUES[epilogue], self._cfg(cfg), self._stream(stream)),
               "fact_linear_grouped_fp8", self._h)
        return out

    def linear_fp8(self, X, W, scale=1.0, bias=None, residual=None, epilogue="NONE", out=None,
                   out_dtype=torch.bfloat16, cfg=None, stream=None):
        """Y = epilogue(scale * X @ W^T)  (fact_linear_fp8).  X [M, K] and W [Nw, K] are FP8 E4M3: torch.float8_e4m3fn
        tensors, or torch.uint8 tensors holding the codes."""
        def codes(t, name):
            if isinstance(t, torch.Tensor) and t.dtype == torch.float8_e4m3fn:
                t = t.view(torch.uint8)
            _need(t, name, torch.uint8, 2)
            return t
        X, W = codes(X, "X"), codes(W, "W")
        M, K = X.shape
        Nw = W.shape[0]
        if W.shape[1] != K:
            raise ValueError("inner dimensions differ")
        if epilogue == "SILU_GATE":
            if Nw % 2:
                raise ValueError("SILU_GATE needs an even number of weight rows")
            N = Nw // 2
        else:
            N = Nw
        if bias is not None:
            _need(bias, "bias", torch.bfloat16, 1)
            if bias.shape[0] != N:
                raise ValueError("bias must have N_out entries")
        if residual is not None:
            _need(residual, "residual", torch.bfloat16, 2)
            if tuple(residual.shape) != (M, N):
                raise ValueError("residual must be [M, N_out]")
        if out is None:
            out = torch.empty((M, N), dtype=out_dtype, device=X.device)
        _need_out(out, (M, N), X)
        nws = self.workspace_bytes("linear_fp8", 1, M, N, K, epilogue, "NK", out.dtype, cfg)
        ws = self.workspace(nws)
        _check(lib().fact_linear_fp8(self._h, M, N, K, _ptr(X), _ld(X), _ptr(W), _ld(W), float(scale), _ptr(bias),
                                     _ptr(residual), _ld(residual) if residual is not None else 0, _ptr(out), _ld(out),
                                     OUT_TYPES[out.dtype], EPILOGUES[epilogue], self._cfg(cfg), _ptr(ws), nws,
                                     self._stream(stream)), "fact_linear_fp8", self._h)
        return out

    def attention(self, q, k, v, causal=True, scale=0.0, out=None, stream=None):
        """O = softmax(scale * Q K^T + causal mask) V  (fact_attention).
        q: [B, Tq, Hq, D], k / v: [B, Tk, Hkv, D] BF16 CUDA tensors (any strides with contiguous head_dim, e.g.
        slices of a fused QKV projection); returns [B, Tq, Hq, D]."""
        for name, t in (("q", q), ("k", k), ("v", v)):
            _need(t, name, torch.bfloat16, 4)
        B, Tq, Hq, D = q.shape
        _, Tk, Hkv, _ = k.shape
        if out is None:
            out = torch.empty((B, Tq, Hq, D), dtype=torch.bfloat16, device=q.device)
        _need_out(out, (B, Tq, Hq, D), q)
        st = lambda t: (int(t.stride(0)), int(t.stride(1)), int(t.stride(2)))
        _check(lib().fact_attention(self._h, B, Tq, Tk, Hq, Hkv, D, _ptr(q), *st(q), _ptr(k), *st(k), _ptr(v), *st(v),
                                    _ptr(out), *st(out), 1 if causal else 0, float(scale), self._stream(stream)),
               "fact_attention", self._h)
        return out

    def norm(self, x, gamma, beta=None, kind="layer", eps=1e-5, out=None, stream=None):
        """Row normalisation (fact_norm): LayerNorm (kind="layer", gamma and beta) or RMSNorm (kind="rms", gamma).
        x: [M, C] BF16 (rows may be strided); returns [M, C]."""
        _need(x, "x", torch.bfloat16, 2)
        M, C = x.shape
        if out is None:
            out = torch.empty((M, C), dtype=torch.bfloat16, device=x.device)
        _check(lib().fact_norm(self._h, NORMS[kind], M, C, _ptr(x), _ld(x), _ptr(gamma), _ptr(beta), float(eps),
                               _ptr(out), _ld(out), self._stream(stream)), "fact_norm", self._h)
        return out

    def block_desc(self, kind, batch, seq, heads_q, heads_kv, head_dim, ffn, weights, eps=1e-5):
        """A fact_block_t for `weights`: a dict of contiguous BF16 CUDA tensors keyed like the struct's pointer
        fields (absent or None = NULL).  The dict must outlive the calls that use the descriptor."""
        b = Block()
        b.kind = BLOCK_KINDS[kind]
        b.batch, b.seq, b.hidden = batch, seq, heads_q * head_dim
        b.heads_q, b.heads_kv, b.head_dim, b.ffn = heads_q, heads_kv, head_dim, ffn
        b.eps = eps
        for name in ("norm1_gamma", "norm1_beta", "wqkv", "bqkv", "wo", "bo", "norm2_gamma", "norm2_beta", "w1",
                     "b1", "w2", "b2"):
            t = weights.get(name)
            if t is not None and not t.is_contiguous():
                raise ValueError(f"{name} must be contiguous")
            setattr(b, name, None if t is None else int(t.data_ptr()))
        return b

    def block_forward(self, desc, x, out=None, workspace=None, stream=None):
        """One transformer block forward (fact_block_forward).  x: [batch * seq, hidden] BF16, contiguous."""
        _need(x, "x", torch.bfloat16, 2)
        if not x.is_contiguous():
            raise ValueError("x must be contiguous")
        if out is None:
            out = torch.empty_like(x)
        need = int(lib().fact_block_workspace_bytes(byref(desc)))
        if workspace is None:
            workspace = self.workspace(need)
        _check(lib().fact_block_forward(self._h, byref(desc), _ptr(x), _ptr(out), _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), self._stream(stream)),
               "fact_block_forward", self._h)
        return out

    def block_intermediates(self, desc, workspace):
        """Views of the intermediates a block_forward call left in `workspace` (fact_block_workspace_offsets):
        dict n (= n2), qkv, a, x1, h, each [tokens, columns] BF16."""
        off = (c_size_t * 5)()
        _check(lib().fact_block_workspace_offsets(byref(desc), off), "fact_block_workspace_offsets")
        tok = int(desc.batch * desc.seq)
        cols = {"n": desc.hidden, "qkv": (desc.heads_q + 2 * desc.heads_kv) * desc.head_dim, "a": desc.hidden,
                "x1": desc.hidden, "h": desc.ffn}
        out = {}
        for i, name in enumerate(("n", "qkv", "a", "x1", "h")):
            nbytes = tok * int(cols[name]) * 2
            out[name] = workspace[int(off[i]): int(off[i]) + nbytes].view(torch.bfloat16).view(tok, int(cols[name]))
        return out

    def tune(self, op, A, B, layout="KN", bias=None, residual=None, epilogue="NONE", out=None,
             out_dtype=torch.bfloat16, workspace_bytes=256 << 20, warmup=0, iters=0, stream=None, cold_l2=False,
             verify=True, inject_fault=-1, records=False):
        """Search tile configurations for this problem on the device (fact_tune_ex): every candidate is verified
        against the default configuration's output, then timed (cold_l2: with L2 overwritten before each launch).
        Returns (Config, best_ms, n_tried), plus the per-candidate records (a list of dicts) with records=True."""
        batched = A.ndim == 3
        batch = A.shape[0] if batched else 1
        M, K = A.shape[-2:]
        Nw = B.shape[-1] if layout == "KN" else B.shape[-2]
        N = Nw // 2 if epilogue == "SILU_GATE" else Nw
        if out is None:
            out = torch.empty(((batch, M, N) if batched else (M, N)), dtype=out_dtype, device=A.device)
        _need_out(out, (batch, M, N) if batched else (M, N), A)
        ws = self.workspace(workspace_bytes)
        best, ms, n = Config(), c_double(0.0), c_int(0)
        self._ws_cache.clear()
        cap = 512
        recs = (TuneRecord * cap)()
        n_recs = c_int(0)
        opts = TuneOpts(1 if cold_l2 else 0, 1 if verify else 0, int(inject_fault), recs, cap, ctypes.pointer(n_recs))
        _check(lib().fact_tune_ex(self._h, OPS[op], batch, M, N, K, _ptr(A), _ld(A), A.stride(0) if batched else 0,
                                  _ptr(B), _ld(B), B.stride(0) if batched else 0, LAYOUTS[layout], _ptr(bias),
                                  _ptr(residual), _ld(residual) if residual is not None else 0,
                                  residual.stride(0) if (residual is not None and batched) else 0, _ptr(out), _ld(out),
                                  out.stride(0) if batched else 0, OUT_TYPES[out.dtype], EPILOGUES[epilogue], _ptr(ws),
                                  ws.numel() if ws is not None else 0, warmup, iters, self._stream(stream),
                                  byref(opts), byref(best), byref(ms), byref(n)), "fact_tune_ex", self._h)
        if records:
            return best, float(ms.value), int(n.value), [recs[i].as_dict() for i in range(min(cap, n_recs.value))]
        return best, float(ms.value), int(n.value)
