"""Python binding of the LoCoCo C ABI (include/lococo.h).

Argument marshalling only: torch supplies device memory and the current stream;
every step of the path runs inside liblococo.so.  Importing this module loads
the library and raises if it has not been built - there is no fallback.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_LIB_PATH = Path(__file__).resolve().parent / "liblococo.so"
if not _LIB_PATH.exists():
    raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2406_05317_b200.build` "
                      "(nvcc, sm_100a). The CUDA library is the only implementation of this path.")
_lib = ctypes.CDLL(str(_LIB_PATH))

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED_SHAPE, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)
F32, BF16 = 0, 1
PATH_AUTO, PATH_SIMT, PATH_TENSOR, PATH_TENSOR_PERSISTENT = 0, 1, 2, 3


class Config(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("M", ctypes.c_int32), ("k", ctypes.c_int32), ("c_in", ctypes.c_int32),
                ("weights_per_head", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("softmax_scale", ctypes.c_float), ("norm_eps", ctypes.c_float),
                ("max_chunk", ctypes.c_int32), ("path", ctypes.c_int32)]


class Tensor(ctypes.Structure):
    _fields_ = [("ptr", ctypes.c_void_p), ("stride_batch", ctypes.c_int64), ("stride_head", ctypes.c_int64),
                ("stride_token", ctypes.c_int64)]


_P, _T, _I = ctypes.c_void_p, Tensor, ctypes.c_int32
_SIGNATURES = {
    "lococo_create": [ctypes.POINTER(Config), ctypes.POINTER(_P)],
    "lococo_destroy": [_P],
    "lococo_workspace_bytes": [_P, ctypes.POINTER(ctypes.c_size_t)],
    "lococo_set_workspace": [_P, _P, ctypes.c_size_t, _P],
    "lococo_set_weights": [_P, _P, _P, _P],
    "lococo_set_protected_slots": [_P, _I],
    "lococo_compress_step": [_P, _T, _T, _I, _T, _T, _I, _T, _T, ctypes.POINTER(_I), _P, _P],
    "lococo_chunk_attention": [_P, _T, _T, _T, _I, _T, _T, _I, _T, _P, _P],
    "lococo_saved_bytes": [_P, _I, _I, ctypes.POINTER(ctypes.c_size_t)],
    "lococo_process_sequence": [_P, _T, _T, _T, _I, _I, _T, _T, _T, ctypes.POINTER(_I), _P, _P],
    "lococo_host_staging_bytes": [_P, _I, ctypes.POINTER(ctypes.c_size_t)],
    "lococo_process_sequence_host": [_P, _P, _P, _P, _I, _I, _P, _P, _P, ctypes.POINTER(_I), _P, ctypes.c_size_t, _P],
    "lococo_backward_scratch_bytes": [_P, _I, _I, ctypes.POINTER(ctypes.c_size_t)],
    "lococo_process_sequence_backward": [_P, _T, _T, _T, _T, _I, _I, _I, _P, _T, _T, _T, _T, _T, _T, _P, _P, _T, _T,
                                         _P, ctypes.c_size_t, _P],
    "lococo_get_last_device_status": [_P, ctypes.POINTER(_I), _P],
    "lococo_launch_count": [_P, ctypes.POINTER(ctypes.c_int64)],
    "lococo_compress_step_static": [ctypes.POINTER(Config), _P, _P, _T, _T, _I, _T, _T, _I, _T, _T, _P],
    "lococo_static_scratch_limit": [ctypes.POINTER(ctypes.c_size_t)],
    "lococo_profile_enable": [_P, _I],
    "lococo_profile_read": [_P, _I, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int64)],
}
for _name, _args in _SIGNATURES.items():
    _fn = getattr(_lib, _name)
    _fn.argtypes = _args
    _fn.restype = ctypes.c_int
_lib.lococo_status_string.argtypes = [ctypes.c_int]
_lib.lococo_status_string.restype = ctypes.c_char_p


class LococoError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {_lib.lococo_status_string(status).decode()} ({status})")


def _check(status: int, where: str):
    if status != OK:
        raise LococoError(status, where)


def status_string(status: int) -> str:
    return _lib.lococo_status_string(status).decode()


def raw():
    """The loaded ctypes library (for tests that call the C ABI directly)."""
    return _lib


def _view(t: torch.Tensor | None) -> Tensor:
    """[batch, heads, tokens, d] torch tensor -> lococo_tensor (strides in elements)."""
    if t is None:
        return Tensor(None, 0, 0, 0)
    if t.dim() != 4 or t.stride(3) != 1:
        raise ValueError("expected a [batch, heads, tokens, d] tensor with contiguous d")
    return Tensor(t.data_ptr(), t.stride(0), t.stride(1), t.stride(2))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: torch.Tensor | None):
    return None if t is None else t.data_ptr()


def static_scratch_limit() -> int:
    n = ctypes.c_size_t()
    _check(_lib.lococo_static_scratch_limit(ctypes.byref(n)), "lococo_static_scratch_limit")
    return n.value


def compress_step_static(cfg: Config, G, bias, K_cache, V_cache, cache_len, K_chunk, V_chunk, K_out, V_out):
    """Compress step (Algorithm 2 Steps 4-5) that allocates nothing: for callers that may not
    call cudaMalloc, the scratch is a fixed array inside the library. Raises LococoError with
    ERR_WORKSPACE when the problem does not fit that array."""
    _check(_lib.lococo_compress_step_static(ctypes.byref(cfg), G.data_ptr(), _ptr(bias), _view(K_cache),
                                            _view(V_cache), cache_len, _view(K_chunk), _view(V_chunk),
                                            K_chunk.shape[2], _view(K_out), _view(V_out), _stream()),
           "lococo_compress_step_static")


class Lococo:
    """A configured chunk-step context: handle + workspace + conv weights."""

    def __init__(self, batch, heads, head_dim, M, k, max_chunk, dtype=torch.bfloat16, c_in=None,
                 weights_per_head=False, softmax_scale=0.0, norm_eps=1e-6, path=PATH_AUTO, device="cuda"):
        self.torch_dtype = dtype
        self.cfg = Config(batch, heads, head_dim, M, k, c_in if c_in is not None else head_dim,
                          int(bool(weights_per_head)), {torch.float32: F32, torch.bfloat16: BF16}[dtype],
                          float(softmax_scale), float(norm_eps), max_chunk, path)
        self._h = _P()
        _check(_lib.lococo_create(ctypes.byref(self.cfg), ctypes.byref(self._h)), "lococo_create")
        n = ctypes.c_size_t()
        _check(_lib.lococo_workspace_bytes(self._h, ctypes.byref(n)), "lococo_workspace_bytes")
        self.device = torch.device(device)
        self.workspace = torch.empty(n.value + 256, dtype=torch.uint8, device=self.device)
        off = (-self.workspace.data_ptr()) % 256
        self._ws_ptr = self.workspace.data_ptr() + off
        _check(_lib.lococo_set_workspace(self._h, self._ws_ptr, n.value, _stream()), "lococo_set_workspace")
        self.workspace_bytes = n.value

    def __del__(self):
        h = getattr(self, "_h", None)
        if h and _lib is not None:      # at interpreter shutdown the module globals may be gone already
            _lib.lococo_destroy(h)
            self._h = None

    @property
    def handle(self):
        return self._h

    def set_weights(self, G: torch.Tensor, bias: torch.Tensor | None = None):
        """G [heads|1, M, c_in, k] (and bias [heads|1, M]) in the configured dtype."""
        c = self.cfg
        sets = c.heads if c.weights_per_head else 1
        if tuple(G.shape) != (sets, c.M, c.c_in, c.k) or G.dtype != self.torch_dtype or not G.is_contiguous():
            raise ValueError("G must be contiguous [heads|1, M, c_in, k] in the configured dtype")
        if bias is not None and (tuple(bias.shape) != (sets, c.M) or bias.dtype != self.torch_dtype):
            raise ValueError("bias must be [heads|1, M] in the configured dtype")
        _check(_lib.lococo_set_weights(self._h, G.data_ptr(), _ptr(bias), _stream()), "lococo_set_weights")

    def set_protected_slots(self, slots: int):
        """Section 5.2: the first `slots` cache slots keep their entries; the others are compressed."""
        _check(_lib.lococo_set_protected_slots(self._h, int(slots)), "lococo_set_protected_slots")

    def compress_step(self, K_cache, V_cache, cache_len, K_chunk, V_chunk, K_out=None, V_out=None, W_out=None):
        """Algorithm 2 Steps 4-5 (or the fill branch). Returns the new cache length."""
        K_out = K_cache if K_out is None else K_out
        V_out = V_cache if V_out is None else V_out
        new_len = _I()
        _check(_lib.lococo_compress_step(self._h, _view(K_cache), _view(V_cache), cache_len, _view(K_chunk),
                                         _view(V_chunk), K_chunk.shape[2], _view(K_out), _view(V_out),
                                         ctypes.byref(new_len), _ptr(W_out), _stream()), "lococo_compress_step")
        return new_len.value

    def chunk_attention(self, Q, K_cache, V_cache, cache_len, K_chunk, V_chunk, O, lse=None):
        """Algorithm 2 Step 3."""
        _check(_lib.lococo_chunk_attention(self._h, _view(Q), _view(K_cache), _view(V_cache), cache_len,
                                           _view(K_chunk), _view(V_chunk), Q.shape[2], _view(O), _ptr(lse),
                                           _stream()), "lococo_chunk_attention")

    def saved_bytes(self, L, B):
        n = ctypes.c_size_t()
        _check(_lib.lococo_saved_bytes(self._h, L, B, ctypes.byref(n)), "lococo_saved_bytes")
        return n.value

    def process_sequence(self, Q, K, V, B, O, K_cache, V_cache, cache_len=0, saved=None):
        """Algorithm 2 over all tokens of Q, K, V. Returns the final cache length."""
        c = _I(cache_len)
        _check(_lib.lococo_process_sequence(self._h, _view(Q), _view(K), _view(V), Q.shape[2], B, _view(O),
                                            _view(K_cache), _view(V_cache), ctypes.byref(c), _ptr(saved),
                                            _stream()), "lococo_process_sequence")
        return c.value

    def host_staging_bytes(self, L):
        n = ctypes.c_size_t()
        _check(_lib.lococo_host_staging_bytes(self._h, L, ctypes.byref(n)), "lococo_host_staging_bytes")
        return n.value

    def process_sequence_host(self, Q_host, K_host, V_host, B, O_host, staging, K_cache_host=None,
                              V_cache_host=None):
        """Algorithm 2 on (pinned) host tensors [batch, heads, L, d]; copies are part of the call."""
        for t in (Q_host, K_host, V_host, O_host):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("host entry point takes contiguous CPU tensors")
        c = _I(0)
        _check(_lib.lococo_process_sequence_host(self._h, Q_host.data_ptr(), K_host.data_ptr(), V_host.data_ptr(),
                                                 Q_host.shape[2], B, O_host.data_ptr(), _ptr(K_cache_host),
                                                 _ptr(V_cache_host), ctypes.byref(c), staging.data_ptr(),
                                                 staging.numel() * staging.element_size(), _stream()),
               "lococo_process_sequence_host")
        return c.value

    def backward_scratch_bytes(self, L, B):
        n = ctypes.c_size_t()
        _check(_lib.lococo_backward_scratch_bytes(self._h, L, B, ctypes.byref(n)), "lococo_backward_scratch_bytes")
        return n.value

    def process_sequence_backward(self, Q, K, V, O, B, saved, dO, dK_cache_final, dV_cache_final, dQ, dK, dV, dG,
                                  dbias, scratch, cache_len_in=0, dK_cache_in=None, dV_cache_in=None):
        """Gradients through one process_sequence call that started from `cache_len_in` cache rows."""
        _check(_lib.lococo_process_sequence_backward(
            self._h, _view(Q), _view(K), _view(V), _view(O), Q.shape[2], B, cache_len_in, _ptr(saved), _view(dO),
            _view(dK_cache_final), _view(dV_cache_final), _view(dQ), _view(dK), _view(dV), _ptr(dG), _ptr(dbias),
            _view(dK_cache_in), _view(dV_cache_in), scratch.data_ptr(), scratch.numel() * scratch.element_size(),
            _stream()), "lococo_process_sequence_backward")

    def device_status(self) -> int:
        out = _I()
        _check(_lib.lococo_get_last_device_status(self._h, ctypes.byref(out), _stream()),
               "lococo_get_last_device_status")
        return out.value

    def launch_count(self) -> int:
        out = ctypes.c_int64()
        _check(_lib.lococo_launch_count(self._h, ctypes.byref(out)), "lococo_launch_count")
        return out.value

    def profile(self, on: bool):
        """Start (or stop) recording per-kernel CUDA-event timings."""
        _check(_lib.lococo_profile_enable(self._h, int(on)), "lococo_profile_enable")

    def profile_read(self, kind: int):
        """(total milliseconds, launches) of kernel class `kind` (0: conv, 1: attention)."""
        ms, n = ctypes.c_double(), ctypes.c_int64()
        _check(_lib.lococo_profile_read(self._h, kind, ctypes.byref(ms), ctypes.byref(n)), "lococo_profile_read")
        return ms.value, n.value
