"""ctypes binding of include/entropyinfer.h -- same names, argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libentropyinfer.so")


class EiParams(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32),
        ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("seq_len", C.c_int32), ("segment_len", C.c_int32), ("block_len", C.c_int32),
        ("budget_mode", C.c_int32),
        ("q_stride_head", C.c_int64), ("q_stride_tok", C.c_int64),
        ("k_stride_head", C.c_int64), ("k_stride_tok", C.c_int64),
        ("v_stride_head", C.c_int64), ("v_stride_tok", C.c_int64),
        ("o_stride_head", C.c_int64), ("o_stride_tok", C.c_int64),
        ("base_budget_tokens", C.c_double), ("budget_fraction", C.c_double),
        ("entropy_threshold", C.c_double), ("alpha", C.c_double), ("delta_t", C.c_double),
        ("max_mult", C.c_double), ("obs_scale", C.c_double), ("attn_scale", C.c_double),
        ("flags", C.c_uint32), ("q_len", C.c_uint32),
    ]


class EiCompressParams(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32),
        ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("kv_len", C.c_int32), ("window", C.c_int32), ("budget", C.c_int32), ("reserved", C.c_int32),
        ("q_stride_head", C.c_int64), ("q_stride_tok", C.c_int64),
        ("k_stride_head", C.c_int64), ("k_stride_tok", C.c_int64),
        ("v_stride_head", C.c_int64), ("v_stride_tok", C.c_int64),
    ]


STATUS = dict(OK=0, INVALID_ARG=-1, UNSUPPORTED_SHAPE=-2, BUDGET_INFEASIBLE=-3, ARCH=-4, ALLOC=-5,
              CUDA=-6, DEVICE_TIMEOUT=-7, PLAN_MISMATCH=-8, NOT_PLANNED=-9, SCRATCH_TOO_SMALL=-10, WRONG_DEVICE=-11)
ITEM = dict(GROUP_ENTROPY=11, GROUP_SCORES=12, ENTROPY=0, CLASS=1, BUDGET=2, OFFSETS=3, INDICES=4, SCORES=5, QMAX=6, QMIN=7, KMAX=8,
            KMIN=9, STATS=10, MULTIPLIERS=13)
BUDGET_BASE_TOKENS, BUDGET_TOTAL_FRACTION = 0, 1
ROPE_NO_POOL = 1
FLAG_ATTN_P_VIA_SMEM = 1
FLAG_ATTN_SINGLE_TILE = 2
FLAG_ATTN_PAIR_8WARP = 4
FLAG_GROUP_SHARED = 8
FLAG_PLAN_STAGED = 16
FLAG_PLAN_FUSED = 32
FLAG_ATTN_PERSISTENT = 64
FLAG_ATTN_PER_CTA = 128
FLAG_ATTN_NO_SKIP = 256
FLAG_ATTN_SKIP_ZERO_PV = 512
FLAG_ATTN_QUAD = 1024
FLAG_ATTN_SPLIT = 2048
FLAG_ATTN_TRI = 4096
FLAG_HEAD_SHARD = 8192

# every symbol the header declares: (name, restype, argtypes)
_P = C.c_void_p
SYMBOLS = [
    ("ei_params_default", C.c_int, [C.POINTER(EiParams), C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_double]),
    ("ei_plan_create", C.c_int, [C.POINTER(EiParams), C.POINTER(_P)]),
    ("ei_plan_destroy", None, [_P]),
    ("ei_plan", C.c_int, [_P, _P, _P, _P, _P]),
    ("ei_sparse_prefill", C.c_int, [_P, _P, _P, _P, _P, _P]),
    ("ei_prefill_host", C.c_int, [_P, _P, _P, _P, _P, _P]),
    ("ei_prefill_varlen", C.c_int, [_P, _P, _P, _P, _P, C.POINTER(C.c_int32), C.c_int, _P]),
    ("ei_rope_pool", C.c_int, [_P, _P, _P, _P, _P, _P, _P, C.c_uint32, _P]),
    ("ei_plan_pooled", C.c_int, [_P, _P]),
    ("ei_stage_pool", C.c_int, [_P, _P, _P, _P]),
    ("ei_stage_observe", C.c_int, [_P, _P]),
    ("ei_stage_budget", C.c_int, [_P, _P]),
    ("ei_plan_observe", C.c_int, [_P, _P, _P, _P]),
    ("ei_stage_multipliers", C.c_int, [_P, _P, _P]),
    ("ei_stage_apportion", C.c_int, [_P, _P, C.c_int, C.c_int, C.c_int64, _P]),
    ("ei_stage_select", C.c_int, [_P, _P]),
    ("ei_plan_get", C.c_int, [_P, C.c_int, C.POINTER(_P), C.POINTER(C.c_size_t)]),
    ("ei_plan_read", C.c_int, [_P, C.c_int, _P, C.c_size_t, _P]),
    ("ei_plan_write", C.c_int, [_P, C.c_int, _P, C.c_size_t, _P]),
    ("ei_plan_set_lists", C.c_int, [_P, _P, _P, C.c_size_t, _P]),
    ("ei_plan_set_lengths", C.c_int, [_P, C.c_int, C.c_int, C.c_int]),
    ("ei_plan_status", C.c_int, [_P, _P]),
    ("ei_plan_debug_waits", C.c_int, [_P, C.c_int, C.c_int, _P]),
    ("ei_plan_total_blocks", C.c_int64, [_P]),
    ("ei_plan_launches", C.c_int64, [_P]),
    ("ei_entropy_noalloc", C.c_int, [C.POINTER(EiParams), _P, _P, _P, _P]),
    ("ei_latent_compress_workspace_bytes", C.c_size_t, [C.POINTER(EiCompressParams)]),
    ("ei_latent_compress", C.c_int, [C.POINTER(EiCompressParams), _P, _P, _P, _P, _P, _P, _P, _P]),
    ("ei_status_string", C.c_char_p, [C.c_int]),
    ("ei_version", C.c_int, []),
]

_lib = None


class EiError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


def load_library(path: str = LIB_PATH) -> C.CDLL:
    """Load libentropyinfer.so; there is no fallback -- a missing library is an error."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(path) and path == LIB_PATH:
        # a fresh checkout holds sources only: compile them (nvcc, sm_100a; about a minute); nothing else can stand in
        try:
            from . import build as _build
            _build.build()
        except Exception as exc:  # noqa: BLE001
            raise FileNotFoundError(
                f"{path} not found and building it failed ({exc}); build it with "
                "`python -m paper_2606_09508_b200.build` (nvcc, sm_100a); this package has no CPU or eager fallback")
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} not found: build it with `python -m paper_2606_09508_b200.build` "
            "(nvcc, sm_100a); this package has no CPU or eager fallback")
    lib_ = C.CDLL(path)
    for name, res, args in SYMBOLS:
        fn = getattr(lib_, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib_
    return lib_


def lib() -> C.CDLL:
    return load_library()


def status_string(code: int) -> str:
    return lib().ei_status_string(int(code)).decode()


def version() -> int:
    return lib().ei_version()


def _check(code: int, where: str):
    if code != 0:
        raise EiError(code, where)


def params_default(H, Hkv, d, N, L_S, L_B, fraction=0.0) -> EiParams:
    p = EiParams()
    _check(lib().ei_params_default(C.byref(p), H, Hkv, d, N, L_S, L_B, float(fraction)), "ei_params_default")
    return p


_ITEM_DTYPE = {"GROUP_ENTROPY": np.float32, "GROUP_SCORES": np.float32, "ENTROPY": np.float32, "CLASS": np.uint8, "BUDGET": np.int32, "OFFSETS": np.int32,
               "INDICES": np.int32, "SCORES": np.float32, "QMAX": np.uint16, "QMIN": np.uint16,
               "KMAX": np.uint16, "KMIN": np.uint16, "STATS": np.int64, "MULTIPLIERS": np.int32}


def _dev_ptr(t) -> int:
    """Device pointer of a torch CUDA tensor (or a raw integer address)."""
    if isinstance(t, int):
        return t
    if t is None:
        return 0
    assert t.is_cuda, "expected a CUDA tensor"
    return t.data_ptr()


def _stream_ptr(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def entropy_noalloc(params: EiParams, q, k, entropy_out, stream=None):
    """ei_entropy_noalloc: entropy table [H, C_S] (float32 CUDA tensor, caller-owned) without any
    device allocation by the library; for callers whose own allocator owns the device."""
    _check(lib().ei_entropy_noalloc(C.byref(params), _dev_ptr(q), _dev_ptr(k), _dev_ptr(entropy_out),
                                    _stream_ptr(stream)), "ei_entropy_noalloc")


NOALLOC_SCRATCH_BYTES = 32 << 20   # EI_NOALLOC_SCRATCH_BYTES in the header


def compress_params(H, Hkv, d, L, window, budget) -> EiCompressParams:
    """Contiguous q_window [H, window, d], k / v [Hkv, L, d]."""
    p = EiCompressParams()
    p.struct_size = C.sizeof(EiCompressParams)
    p.n_q_heads, p.n_kv_heads, p.head_dim, p.kv_len, p.window, p.budget = H, Hkv, d, L, window, budget
    p.q_stride_tok = p.k_stride_tok = p.v_stride_tok = d
    p.q_stride_head = window * d
    p.k_stride_head = p.v_stride_head = L * d
    return p


def latent_compress_workspace_bytes(params: EiCompressParams) -> int:
    return int(lib().ei_latent_compress_workspace_bytes(C.byref(params)))


def latent_compress(params: EiCompressParams, q_window, k, v, workspace, idx_out, k_out, v_out, stream=None):
    """ei_latent_compress: all arguments are CUDA tensors owned by the caller."""
    _check(lib().ei_latent_compress(C.byref(params), _dev_ptr(q_window), _dev_ptr(k), _dev_ptr(v), _dev_ptr(workspace),
                                    _dev_ptr(idx_out), _dev_ptr(k_out), _dev_ptr(v_out), _stream_ptr(stream)),
           "ei_latent_compress")


class Plan:
    """Owns an ei_plan_t.  Methods mirror the C entry points one to one."""

    def __init__(self, params: EiParams):
        self.params = params
        self._h = _P()
        _check(lib().ei_plan_create(C.byref(params), C.byref(self._h)), "ei_plan_create")
        self.Nq = params.q_len or params.seq_len          # chunked prefill: the queries are the last q_len positions
        self.H, self.C_S = params.n_q_heads, -(-self.Nq // params.segment_len)   # ceil: a short last segment
        self.r = params.segment_len // params.block_len
        self.group_shared = bool(params.flags & FLAG_GROUP_SHARED)
        self.list_heads = params.n_kv_heads if self.group_shared else self.H   # heads that own a block list

    def close(self):
        if self._h:
            lib().ei_plan_destroy(self._h)
            self._h = _P()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the two calls of the path
    def plan(self, q, k, v=None, stream=None):
        _check(lib().ei_plan(self._h, _dev_ptr(q), _dev_ptr(k), _dev_ptr(v), _stream_ptr(stream)), "ei_plan")

    def sparse_prefill(self, q, k, v, out, stream=None):
        _check(lib().ei_sparse_prefill(self._h, _dev_ptr(q), _dev_ptr(k), _dev_ptr(v), _dev_ptr(out),
                                       _stream_ptr(stream)), "ei_sparse_prefill")

    def prefill_host(self, q_host, k_host, v_host, out_host, stream=None):
        """q_host.. are host buffers (numpy arrays or pinned CPU torch tensors, contiguous bf16 bits)."""
        def hp(a):
            return a.ctypes.data if isinstance(a, np.ndarray) else a.data_ptr()
        _check(lib().ei_prefill_host(self._h, hp(q_host), hp(k_host), hp(v_host), hp(out_host),
                                     _stream_ptr(stream)), "ei_prefill_host")

    def rope_pool(self, q_in, k_in, cos, sin, q_out=None, k_out=None, pool=True, stream=None):
        """Rotary embedding of q and k (in place unless q_out / k_out are given) with the pooling folded in."""
        _check(lib().ei_rope_pool(self._h, _dev_ptr(q_in), _dev_ptr(k_in), _dev_ptr(cos), _dev_ptr(sin),
                                  _dev_ptr(q_in if q_out is None else q_out), _dev_ptr(k_in if k_out is None else k_out),
                                  0 if pool else ROPE_NO_POOL, _stream_ptr(stream)), "ei_rope_pool")

    def plan_pooled(self, stream=None):
        """Stages 1b-3 from the representatives the plan holds."""
        _check(lib().ei_plan_pooled(self._h, _stream_ptr(stream)), "ei_plan_pooled")

    def prefill_varlen(self, q, k, v, out, cu_seqlens, stream=None):
        """Packed batch: cu_seqlens (host integers, n_seqs + 1) delimits the sequences along the token axis."""
        cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
        _check(lib().ei_prefill_varlen(self._h, _dev_ptr(q), _dev_ptr(k), _dev_ptr(v), _dev_ptr(out),
                                       cu.ctypes.data_as(C.POINTER(C.c_int32)), int(cu.size) - 1, _stream_ptr(stream)),
               "ei_prefill_varlen")
        last = [int(b - a) for a, b in zip(cu[:-1], cu[1:]) if b > a]
        if last:                                     # the plan is left targeted at the last non-empty sequence
            self.params.seq_len, self.params.q_len = last[-1], 0
            self.Nq = last[-1]
            self.C_S = -(-self.Nq // self.params.segment_len)

    # ---- single stages
    def stage_pool(self, q, k, stream=None):
        _check(lib().ei_stage_pool(self._h, _dev_ptr(q), _dev_ptr(k), _stream_ptr(stream)), "ei_stage_pool")

    def stage_observe(self, stream=None):
        _check(lib().ei_stage_observe(self._h, _stream_ptr(stream)), "ei_stage_observe")

    def stage_budget(self, stream=None):
        _check(lib().ei_stage_budget(self._h, _stream_ptr(stream)), "ei_stage_budget")

    # ---- a layer's heads sharded over several plans (one per GPU)
    def observe(self, q, k, stream=None):
        """Stages 1a + 1b alone."""
        _check(lib().ei_plan_observe(self._h, _dev_ptr(q), _dev_ptr(k), _stream_ptr(stream)), "ei_plan_observe")

    def stage_multipliers(self, out=None, stream=None):
        """Alg. 3's classes and multipliers; `out`: an int32 device tensor [H, C_S] that also receives the table."""
        _check(lib().ei_stage_multipliers(self._h, _dev_ptr(out), _stream_ptr(stream)), "ei_stage_multipliers")

    def stage_apportion(self, multipliers_all, n_heads_all: int, first_head: int, total_all: int, stream=None):
        """Block counts of this plan's heads from the gathered tables of all heads (device int32 [n_heads_all, C_S])."""
        _check(lib().ei_stage_apportion(self._h, _dev_ptr(multipliers_all), int(n_heads_all), int(first_head),
                                        int(total_all), _stream_ptr(stream)), "ei_stage_apportion")

    def stage_select(self, stream=None):
        _check(lib().ei_stage_select(self._h, _stream_ptr(stream)), "ei_stage_select")

    # ---- plan items
    def get(self, item: str):
        ptr, n = _P(), C.c_size_t()
        _check(lib().ei_plan_get(self._h, ITEM[item], C.byref(ptr), C.byref(n)), "ei_plan_get")
        return ptr.value, n.value

    def read(self, item: str, count: int | None = None, stream=None) -> np.ndarray:
        _, nbytes = self.get(item)
        dt = np.dtype(_ITEM_DTYPE[item])
        n = nbytes // dt.itemsize if count is None else count
        out = np.empty(n, dt)
        if n:
            _check(lib().ei_plan_read(self._h, ITEM[item], out.ctypes.data, n * dt.itemsize, _stream_ptr(stream)),
                   "ei_plan_read")
        return out

    def write(self, item: str, arr: np.ndarray, stream=None):
        arr = np.ascontiguousarray(arr, dtype=_ITEM_DTYPE[item])
        _check(lib().ei_plan_write(self._h, ITEM[item], arr.ctypes.data, arr.nbytes, _stream_ptr(stream)),
               "ei_plan_write")

    def set_lists(self, k: np.ndarray, idx: np.ndarray, stream=None):
        k = np.ascontiguousarray(k, dtype=np.int32).ravel()
        idx = np.ascontiguousarray(idx, dtype=np.int32).ravel()
        _check(lib().ei_plan_set_lists(self._h, k.ctypes.data, idx.ctypes.data if idx.size else None, idx.size,
                                       _stream_ptr(stream)), "ei_plan_set_lists")

    def set_lengths(self, seq_len: int, q_len: int = 0, k_blocks_valid: int = 0):
        """Re-target the plan (no allocation) to seq_len keys of which the last q_len are the queries."""
        _check(lib().ei_plan_set_lengths(self._h, int(seq_len), int(q_len), int(k_blocks_valid)), "ei_plan_set_lengths")
        self.params.seq_len, self.params.q_len = int(seq_len), int(q_len)
        self.Nq = q_len or seq_len
        self.C_S = -(-self.Nq // self.params.segment_len)

    def status(self, stream=None) -> int:
        return lib().ei_plan_status(self._h, _stream_ptr(stream))

    def debug_waits(self, wait_limit_log2: int = 0, skip_ring_item: int = -1, stream=None):
        """Testing aid: shorten the device-side wait bound and / or make the producer leave out one K/V load."""
        _check(lib().ei_plan_debug_waits(self._h, int(wait_limit_log2), int(skip_ring_item), _stream_ptr(stream)),
               "ei_plan_debug_waits")

    def total_blocks(self) -> int:
        return lib().ei_plan_total_blocks(self._h)

    def launches(self) -> int:
        return lib().ei_plan_launches(self._h)

    # ---- convenience: everything the planner produced, on the host
    def results(self, stream=None) -> dict:
        cells = self.list_heads * self.C_S
        offsets = self.read("OFFSETS", stream=stream)
        total = int(offsets[cells])
        extra = {}
        if self.group_shared:
            extra["group_entropy"] = self.read("GROUP_ENTROPY", stream=stream).reshape(self.list_heads, self.C_S)
        return dict(
            entropy=self.read("ENTROPY", stream=stream).reshape(self.H, self.C_S),
            rigid=self.read("CLASS", stream=stream),
            k=self.read("BUDGET", stream=stream).reshape(self.list_heads, self.C_S),
            **extra,
            offsets=offsets,
            idx=self.read("INDICES", count=total, stream=stream),
            stats=self.read("STATS", stream=stream),
        )
