from __future__ import annotations

import ctypes
from ctypes import POINTER, c_char_p, c_float, c_int32, c_int64, c_size_t, c_void_p
from dataclasses import dataclass
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_LIB_PATH = _HERE / "libpsa.so"
_lib = None

PSA_OUT_BF16, PSA_OUT_F32 = 0, 1

# every symbol include/psa.h declares
EXPORTED_SYMBOLS = [
    "psa_plan_create", "psa_plan_create_cascade", "psa_plan_create_prefill", "psa_prefill", "psa_plan_destroy", "psa_plan_get_info", "psa_plan_workspace_bytes",
    "psa_plan_bind_workspace", "psa_plan_prefix_items", "psa_plan_suffix_items",
    "psa_decode", "psa_decode_static", "psa_static_check_status", "psa_static_selftest_bounded_wait", "psa_decode_prefix", "psa_decode_suffix", "psa_decode_merge",
    "psa_decode_host_staging_bytes", "psa_decode_host", "psa_check_status", "psa_selftest_bounded_wait", "psa_append_kv", "psa_append_kv_alloc", "psa_validate_page_table", "psa_sample_scratch_bytes", "psa_sample_tokens", "psa_sample_tokens_at", "psa_attn_task",
    "psa_status_string", "psa_last_error_message", "psa_version",
]


class PsaError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"psa status {status} ({status_string(status)}): {message}")
        self.status = status


class _Config(ctypes.Structure):
    _fields_ = [("num_q_heads", c_int32), ("num_kv_heads", c_int32), ("head_dim", c_int32), ("page_size", c_int32),
                ("sm_scale", c_float), ("out_dtype", c_int32), ("num_sms", c_int32), ("suffix_chunk_tokens", c_int32),
                ("prefix_tiles_per_item", c_int32), ("prefix_rows_per_item", c_int32), ("prefix_kernel", c_int32)]


class _Info(ctypes.Structure):
    _fields_ = [("num_sms", c_int32), ("num_samples", c_int32), ("num_prefix_items", c_int32),
                ("num_suffix_items", c_int32), ("prefix_tile_keys", c_int32), ("prefix_tiles_per_item", c_int32),
                ("suffix_chunk_tokens", c_int32), ("kernel_launches", c_int32), ("num_partial_rows", c_int64)]


@dataclass
class PlanInfo:
    num_sms: int
    num_samples: int
    num_prefix_items: int
    num_suffix_items: int
    prefix_tile_keys: int
    prefix_tiles_per_item: int
    suffix_chunk_tokens: int
    kernel_launches: int
    num_partial_rows: int


def library_path() -> Path:
    return _LIB_PATH


def library():
    """Load libpsa.so.  Raises if it has not been built: there is no other implementation."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2502_02534_b200.build`")
        lib = ctypes.CDLL(str(_LIB_PATH))
        P = c_void_p
        lib.psa_plan_create.restype = c_int32
        lib.psa_plan_create.argtypes = [POINTER(_Config), c_int32, P, P, P, POINTER(c_void_p)]
        lib.psa_plan_create_cascade.restype = c_int32
        lib.psa_plan_create_cascade.argtypes = [POINTER(_Config), c_int32, P, P, P, c_int32, P, POINTER(c_void_p)]
        lib.psa_plan_create_prefill.restype = c_int32
        lib.psa_plan_create_prefill.argtypes = [POINTER(_Config), c_int32, P, POINTER(c_void_p)]
        lib.psa_prefill.restype = c_int32
        lib.psa_prefill.argtypes = [P, P, P, P, POINTER(c_int64), P, P, P, c_size_t, P]
        lib.psa_plan_destroy.restype = c_int32
        lib.psa_plan_destroy.argtypes = [P]
        lib.psa_plan_get_info.restype = c_int32
        lib.psa_plan_get_info.argtypes = [P, POINTER(_Info)]
        lib.psa_plan_workspace_bytes.restype = c_size_t
        lib.psa_plan_workspace_bytes.argtypes = [P]
        lib.psa_plan_bind_workspace.restype = c_int32
        lib.psa_plan_bind_workspace.argtypes = [P, P, c_size_t, P]
        lib.psa_plan_prefix_items.restype = c_int32
        lib.psa_plan_prefix_items.argtypes = [P, P]
        lib.psa_plan_suffix_items.restype = c_int32
        lib.psa_plan_suffix_items.argtypes = [P, P]
        lib.psa_decode.restype = c_int32
        lib.psa_decode.argtypes = [P, P, P, P, POINTER(c_int64), P, P, POINTER(c_int64), P, P, P, P, P, P, c_size_t, P]
        lib.psa_decode_static.restype = c_int32
        lib.psa_decode_static.argtypes = [P, P, P, P, POINTER(c_int64), P, P, POINTER(c_int64), P, P, P, P, P, P]
        lib.psa_static_check_status.restype = c_int32
        lib.psa_static_check_status.argtypes = [P]
        lib.psa_static_selftest_bounded_wait.restype = c_int32
        lib.psa_static_selftest_bounded_wait.argtypes = [ctypes.c_uint64, P]
        lib.psa_decode_prefix.restype = c_int32
        lib.psa_decode_prefix.argtypes = [P, P, P, P, POINTER(c_int64), P, c_size_t, P]
        lib.psa_decode_suffix.restype = c_int32
        lib.psa_decode_suffix.argtypes = [P, P, P, P, POINTER(c_int64), P, P, P, P, c_size_t, P]
        lib.psa_decode_merge.restype = c_int32
        lib.psa_decode_merge.argtypes = [P, P, P, P, P, c_size_t, P]
        lib.psa_decode_host_staging_bytes.restype = c_size_t
        lib.psa_decode_host_staging_bytes.argtypes = [P, c_int64, c_int64, c_int64]
        lib.psa_decode_host.restype = c_int32
        lib.psa_decode_host.argtypes = [P, P, P, P, c_int64, P, P, c_int64, P, P, c_int64, P, P, P, P, c_size_t, P, c_size_t, P]
        lib.psa_check_status.restype = c_int32
        lib.psa_check_status.argtypes = [P, P, P]
        lib.psa_append_kv.restype = c_int32
        lib.psa_append_kv.argtypes = [P, P, P, P, P, POINTER(c_int64), P, P, P, P, c_size_t, P]
        lib.psa_append_kv_alloc.restype = c_int32
        lib.psa_append_kv_alloc.argtypes = [P, P, P, P, P, POINTER(c_int64), P, P, P, P, P, P, c_size_t, P]
        lib.psa_sample_tokens_at.restype = c_int32
        lib.psa_sample_tokens_at.argtypes = [P, c_int32, c_int64, c_int32, c_int32, P, P, P, ctypes.c_uint32, P, P, c_size_t, P]
        lib.psa_validate_page_table.restype = c_int32
        lib.psa_validate_page_table.argtypes = [P, P, P, P, c_int64, P, c_size_t, P]
        lib.psa_sample_scratch_bytes.restype = c_size_t
        lib.psa_sample_scratch_bytes.argtypes = [c_int32]
        lib.psa_sample_tokens.restype = c_int32
        lib.psa_sample_tokens.argtypes = [P, c_int32, c_int64, c_int32, c_int32, P, P, ctypes.c_uint32, P, P, c_size_t, P]
        lib.psa_attn_task.restype = c_int32
        lib.psa_attn_task.argtypes = [c_int32, P, P, P, c_int32, c_int32, c_int32, c_float, P, P, P, P]
        lib.psa_selftest_bounded_wait.restype = c_int32
        lib.psa_selftest_bounded_wait.argtypes = [P, c_size_t, ctypes.c_uint64, P]
        lib.psa_status_string.restype = c_char_p
        lib.psa_status_string.argtypes = [c_int32]
        lib.psa_last_error_message.restype = c_char_p
        lib.psa_last_error_message.argtypes = []
        lib.psa_version.restype = c_int32
        lib.psa_version.argtypes = []
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return library().psa_status_string(int(status)).decode()


def _check(status: int):
    if status != 0:
        raise PsaError(status, library().psa_last_error_message().decode())


def _ptr(t):
    """Address of a torch tensor / numpy array / None."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream_ptr(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


class Plan:
    """psa_plan_create / psa_plan_destroy, plus the workspace the plan needs (a torch uint8 tensor)."""

    def __init__(self, prefix_lens, n_samples_per_prefix, suffix_lens, *, num_q_heads, num_kv_heads, head_dim,
                 page_size=16, sm_scale=None, out_dtype="bf16", num_sms=0, suffix_chunk_tokens=0, prefix_tiles_per_item=0,
                 prefix_rows_per_item=0, prefix_kernel=0, groups=None, prefill_prompt_lens=None):
        """``groups`` = (first_sample[], n_samples[], token_len[]) plans a cascade of shared prefixes
        (psa_plan_create_cascade); ``prefix_lens`` / ``n_samples_per_prefix`` are then ignored."""
        lib = library()
        self.prefix_lens, self.n_samples, self.suffix_len_bounds = _i32(prefix_lens), _i32(n_samples_per_prefix), _i32(suffix_lens)
        self.num_q_heads, self.num_kv_heads, self.head_dim, self.page_size = num_q_heads, num_kv_heads, head_dim, page_size
        self.sm_scale = float(sm_scale if sm_scale is not None else head_dim ** -0.5)
        self.out_dtype = {"bf16": PSA_OUT_BF16, "f32": PSA_OUT_F32}[out_dtype]
        cfg = _Config(num_q_heads, num_kv_heads, head_dim, page_size, self.sm_scale, self.out_dtype, num_sms,
                      suffix_chunk_tokens, prefix_tiles_per_item, prefix_rows_per_item, int(prefix_kernel))
        handle = c_void_p()
        self._h = None
        if prefill_prompt_lens is not None:     # causal self-attention of whole prompts (psa_plan_create_prefill)
            self.prompt_lens = _i32(prefill_prompt_lens)
            _check(lib.psa_plan_create_prefill(ctypes.byref(cfg), len(self.prompt_lens), _ptr(self.prompt_lens), ctypes.byref(handle)))
        elif groups is None:
            _check(lib.psa_plan_create(ctypes.byref(cfg), len(self.prefix_lens), _ptr(self.prefix_lens), _ptr(self.n_samples),
                                       _ptr(self.suffix_len_bounds), ctypes.byref(handle)))
        else:
            self.groups = tuple(_i32(a) for a in groups)
            _check(lib.psa_plan_create_cascade(ctypes.byref(cfg), len(self.groups[0]), _ptr(self.groups[0]), _ptr(self.groups[1]),
                                               _ptr(self.groups[2]), len(self.suffix_len_bounds), _ptr(self.suffix_len_bounds),
                                               ctypes.byref(handle)))
        self._h = handle
        self.workspace = None

    def __del__(self):
        if getattr(self, "_h", None):
            try:
                library().psa_plan_destroy(self._h)
            except Exception:       # interpreter shutdown: the module globals are already gone
                pass
            self._h = None

    @property
    def handle(self):
        return self._h

    @property
    def info(self) -> PlanInfo:
        i = _Info()
        _check(library().psa_plan_get_info(self._h, ctypes.byref(i)))
        return PlanInfo(*(getattr(i, f[0]) for f in _Info._fields_))

    @property
    def workspace_bytes(self) -> int:
        return int(library().psa_plan_workspace_bytes(self._h))

    def prefix_items(self) -> np.ndarray:
        n = library().psa_plan_prefix_items(self._h, None)
        a = np.zeros((n, 8), dtype=np.int32)
        library().psa_plan_prefix_items(self._h, _ptr(a))
        return a

    def suffix_items(self) -> np.ndarray:
        n = library().psa_plan_suffix_items(self._h, None)
        a = np.zeros((n, 4), dtype=np.int32)
        library().psa_plan_suffix_items(self._h, _ptr(a))
        return a

    def bind_workspace(self, workspace=None, stream=None):
        """Allocate (through torch) or adopt a device workspace and upload the work lists into it."""
        import torch
        if workspace is None:
            workspace = torch.empty(max(256, self.workspace_bytes), dtype=torch.uint8, device="cuda")
        _check(library().psa_plan_bind_workspace(self._h, _ptr(workspace), workspace.numel(), _stream_ptr(stream)))
        self.workspace = workspace
        return workspace

    def validate_page_table(self, page_indptr, page_indices, suffix_lens, num_pool_pages, stream=None):
        """psa_validate_page_table: enqueue the check; check_status() raises PSA_ERR_BOUNDS if the table is bad."""
        if self.workspace is None:
            self.bind_workspace(stream=stream)
        _check(library().psa_validate_page_table(self._h, _ptr(page_indptr), _ptr(page_indices), _ptr(suffix_lens),
                                                 int(num_pool_pages), _ptr(self.workspace), self.workspace.numel(), _stream_ptr(stream)))

    def selftest_bounded_wait(self, limit_ns=2_000_000, stream=None):
        """Enqueue the kernel whose wait can never be satisfied; check_status() must then raise PSA_ERR_TIMEOUT."""
        _check(library().psa_selftest_bounded_wait(_ptr(self.workspace), self.workspace.numel(), int(limit_ns), _stream_ptr(stream)))

    def check_status(self, stream=None):
        _check(library().psa_check_status(self._h, _ptr(self.workspace), _stream_ptr(stream)))


def _strides(values, n):
    arr = (c_int64 * n)(*[int(v) for v in values])
    return arr


def default_prefix_strides(plan: Plan):
    return (plan.num_kv_heads * plan.head_dim, plan.head_dim)


def default_pool_strides(plan: Plan):
    return (plan.num_kv_heads * plan.page_size * plan.head_dim, plan.page_size * plan.head_dim, plan.head_dim)


def decode(plan: Plan, q, prefix_k, prefix_v, suffix_k_pool, suffix_v_pool, page_indptr, page_indices, suffix_lens,
           out, lse, *, prefix_strides=None, pool_strides=None, stream=None, stage="all"):
    """psa_decode (or one of its stages) on torch CUDA tensors.  Only enqueues work."""
    lib = library()
    if plan.workspace is None:
        plan.bind_workspace(stream=stream)
    ws, wsb, st = _ptr(plan.workspace), plan.workspace.numel(), _stream_ptr(stream)
    pst = _strides(prefix_strides or default_prefix_strides(plan), 2)
    qst = _strides(pool_strides or default_pool_strides(plan), 3)
    if stage == "all":
        _check(lib.psa_decode(plan.handle, _ptr(q), _ptr(prefix_k), _ptr(prefix_v), pst, _ptr(suffix_k_pool),
                              _ptr(suffix_v_pool), qst, _ptr(page_indptr), _ptr(page_indices), _ptr(suffix_lens),
                              _ptr(out), _ptr(lse), ws, wsb, st))
    elif stage == "prefix":
        _check(lib.psa_decode_prefix(plan.handle, _ptr(q), _ptr(prefix_k), _ptr(prefix_v), pst, ws, wsb, st))
    elif stage == "suffix":
        _check(lib.psa_decode_suffix(plan.handle, _ptr(q), _ptr(suffix_k_pool), _ptr(suffix_v_pool), qst,
                                     _ptr(page_indptr), _ptr(page_indices), _ptr(suffix_lens), ws, wsb, st))
    elif stage == "merge":
        _check(lib.psa_decode_merge(plan.handle, _ptr(suffix_lens), _ptr(out), _ptr(lse), ws, wsb, st))
    else:
        raise ValueError(stage)


STATIC_WORKSPACE_BYTES = 16 << 20


def decode_static(plan: Plan, q, prefix_k, prefix_v, suffix_k_pool, suffix_v_pool, page_indptr, page_indices,
                  suffix_lens, out, lse, *, prefix_strides=None, pool_strides=None, stream=None):
    """psa_decode_static: the same step with the library's built-in scratch array instead of a
    workspace tensor -- nothing is allocated, here or in the library.  Calls that may overlap on
    the GPU share that array and must be serialised by the caller."""
    pst = _strides(prefix_strides or default_prefix_strides(plan), 2)
    qst = _strides(pool_strides or default_pool_strides(plan), 3)
    _check(library().psa_decode_static(plan.handle, _ptr(q), _ptr(prefix_k), _ptr(prefix_v), pst, _ptr(suffix_k_pool),
                                       _ptr(suffix_v_pool), qst, _ptr(page_indptr), _ptr(page_indices),
                                       _ptr(suffix_lens), _ptr(out), _ptr(lse), _stream_ptr(stream)))


def static_check_status(stream=None):
    """psa_static_check_status: raise if the last psa_decode_static step left a device-side error; clears it."""
    _check(library().psa_static_check_status(_stream_ptr(stream)))


def static_selftest_bounded_wait(limit_ns=2_000_000, stream=None):
    """psa_static_selftest_bounded_wait: the unsatisfiable wait, reporting into the library's own array."""
    _check(library().psa_static_selftest_bounded_wait(int(limit_ns), _stream_ptr(stream)))


def prefill(plan: Plan, q, k, v, out, lse, *, kv_strides=None, stream=None):
    """psa_prefill on torch CUDA tensors: causal attention of every prompt over itself."""
    if plan.workspace is None:
        plan.bind_workspace(stream=stream)
    st = _strides(kv_strides or default_prefix_strides(plan), 2)
    _check(library().psa_prefill(plan.handle, _ptr(q), _ptr(k), _ptr(v), st, _ptr(out), _ptr(lse), _ptr(plan.workspace),
                                 plan.workspace.numel(), _stream_ptr(stream)))


def append_kv(plan: Plan, new_k, new_v, suffix_k_pool, suffix_v_pool, page_indptr, page_indices, suffix_lens, *,
              pool_strides=None, stream=None):
    """psa_append_kv: one new token per sample goes to position suffix_lens[s]; suffix_lens is incremented in place."""
    if plan.workspace is None:
        plan.bind_workspace(stream=stream)
    qst = _strides(pool_strides or default_pool_strides(plan), 3)
    _check(library().psa_append_kv(plan.handle, _ptr(new_k), _ptr(new_v), _ptr(suffix_k_pool), _ptr(suffix_v_pool), qst,
                                   _ptr(page_indptr), _ptr(page_indices), _ptr(suffix_lens), _ptr(plan.workspace),
                                   plan.workspace.numel(), _stream_ptr(stream)))


def append_kv_alloc(plan: Plan, new_k, new_v, suffix_k_pool, suffix_v_pool, page_indptr, page_indices, suffix_lens,
                    free_pages, free_count, *, pool_strides=None, stream=None):
    """psa_append_kv_alloc: like append_kv, but a sample that starts a new page takes it from the stack
    free_pages[0 .. free_count) (int32 device tensors; free_count has one element and is updated in place)."""
    if plan.workspace is None:
        plan.bind_workspace(stream=stream)
    qst = _strides(pool_strides or default_pool_strides(plan), 3)
    _check(library().psa_append_kv_alloc(plan.handle, _ptr(new_k), _ptr(new_v), _ptr(suffix_k_pool), _ptr(suffix_v_pool), qst,
                                         _ptr(page_indptr), _ptr(page_indices), _ptr(suffix_lens), _ptr(free_pages),
                                         _ptr(free_count), _ptr(plan.workspace), plan.workspace.numel(), _stream_ptr(stream)))


def sample_tokens_at(logits, temperature, seeds, step_device, advance=1, tokens=None, scratch=None, *, stream=None):
    """psa_sample_tokens_at: the decode step is read from (and advanced in) the one-element int32 device tensor
    `step_device`, so that a captured graph holding this call can be replayed step after step."""
    import torch
    lib = library()
    B, V = logits.shape
    dtype = {torch.bfloat16: PSA_OUT_BF16, torch.float32: PSA_OUT_F32}[logits.dtype]
    if logits.stride(1) != 1:
        raise ValueError("logits must be contiguous along the vocabulary")
    if tokens is None:
        tokens = torch.empty(B, dtype=torch.int32, device=logits.device)
    if scratch is None:
        scratch = torch.empty(max(8, int(lib.psa_sample_scratch_bytes(B))), dtype=torch.uint8, device=logits.device)
    _check(lib.psa_sample_tokens_at(_ptr(logits), dtype, logits.stride(0), B, V, _ptr(temperature), _ptr(seeds), _ptr(step_device),
                                    int(advance), _ptr(tokens), _ptr(scratch), scratch.numel(), _stream_ptr(stream)))
    return tokens


def sample_tokens(logits, temperature, seeds, step, tokens=None, scratch=None, *, stream=None):
    """psa_sample_tokens on torch CUDA tensors: logits [B, V] (bf16 or f32, rows may be padded: stride(0) >= V),
    temperature [B] f32, seeds [B] int64 (bit pattern of the u64 seed).  Returns the int32 token tensor."""
    import torch
    lib = library()
    B, V = logits.shape
    dtype = {torch.bfloat16: PSA_OUT_BF16, torch.float32: PSA_OUT_F32}[logits.dtype]
    if logits.stride(1) != 1:
        raise ValueError("logits must be contiguous along the vocabulary")
    if tokens is None:
        tokens = torch.empty(B, dtype=torch.int32, device=logits.device)
    need = int(lib.psa_sample_scratch_bytes(B))
    if scratch is None:
        scratch = torch.empty(max(8, need), dtype=torch.uint8, device=logits.device)
    _check(lib.psa_sample_tokens(_ptr(logits), dtype, logits.stride(0), B, V, _ptr(temperature), _ptr(seeds), int(step) & 0xFFFFFFFF,
                                 _ptr(tokens), _ptr(scratch), scratch.numel(), _stream_ptr(stream)))
    return tokens


def attn_task(task, q, k, v, sm_scale, *, stream=None):
    """psa_attn_task on torch CUDA tensors: q [R, D], k / v [M, D] bf16.  Returns (out [R, D] f32, m [R], l [R])."""
    import torch
    R, D = q.shape
    M = k.shape[0]
    out = torch.empty((R, D), dtype=torch.float32, device=q.device)
    m = torch.empty(R, dtype=torch.float32, device=q.device)
    l = torch.empty(R, dtype=torch.float32, device=q.device)
    _check(library().psa_attn_task(int(task), _ptr(q), _ptr(k) if M else None, _ptr(v) if M else None, R, M, D, float(sm_scale),
                                   _ptr(out), _ptr(m), _ptr(l), _stream_ptr(stream)))
    return out, m, l


def decode_host(plan: Plan, q, prefix_k, prefix_v, suffix_k_pool, suffix_v_pool, page_indptr, page_indices, suffix_lens,
                out, lse, staging, *, stream=None):
    """psa_decode_host: every tensor is a host buffer (numpy array or pinned torch CPU tensor)."""
    lib = library()
    if plan.workspace is None:
        plan.bind_workspace(stream=stream)
    n_tok = int(prefix_k.shape[0]) if prefix_k is not None else 0
    n_pages = int(suffix_k_pool.shape[0]) if suffix_k_pool is not None else 0
    n_idx = int(page_indices.shape[0]) if page_indices is not None else 0
    _check(lib.psa_decode_host(plan.handle, _ptr(q), _ptr(prefix_k), _ptr(prefix_v), n_tok, _ptr(suffix_k_pool),
                               _ptr(suffix_v_pool), n_pages, _ptr(page_indptr), _ptr(page_indices), n_idx,
                               _ptr(suffix_lens), _ptr(out), _ptr(lse), _ptr(staging), staging.numel(),
                               _ptr(plan.workspace), plan.workspace.numel(), _stream_ptr(stream)))


def host_staging_bytes(plan: Plan, n_prefix_tokens: int, n_pool_pages: int, n_page_indices: int) -> int:
    return int(library().psa_decode_host_staging_bytes(plan.handle, n_prefix_tokens, n_pool_pages, n_page_indices))
