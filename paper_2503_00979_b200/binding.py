"""Thin ctypes binding of ``libmkv.so`` (``include/mkv.h``): argument marshalling only.

Every function below has the name of the C entry point it calls.  ``MorphKV`` is a small
convenience holder of a context plus the torch tensor that backs its workspace.  PyTorch is
used for device memory and streams; every step of the decode path runs in the library's
CUDA kernels.  There is no fallback: if the library is missing or the call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmkv.so")

OK, INVALID_ARG, BAD_STATE, OOM, CUDA, UNSUPPORTED, DEVICE_TIMEOUT = range(7)
STATUS_NAMES = ["MKV_OK", "MKV_INVALID_ARG", "MKV_BAD_STATE", "MKV_OOM", "MKV_CUDA", "MKV_UNSUPPORTED",
                "MKV_DEVICE_TIMEOUT"]
FUSION = {"sum": 0, "max": 1}
DTYPE = {"bf16": 0, "f32": 1}
KERNEL = {"auto": 0, "simt": 1, "tc": 2}
NORM = {"frozen": 0, "current": 1}
PROFILE = {"recompute": 0, "stored": 1}

EXPORTS = [
    "mkv_default_params", "mkv_workspace_bytes", "mkv_create", "mkv_create_ex", "mkv_destroy", "mkv_reset", "mkv_prefill",
    "mkv_prefill_static", "mkv_prefill_ragged", "mkv_row_state",
    "mkv_decode_step", "mkv_decode_step_layer", "mkv_decode_steps", "mkv_decode_step_host", "mkv_cache_view", "mkv_sync", "mkv_last_error",
    "mkv_launch_count", "mkv_kernel_name",
]


class mkv_params(C.Structure):
    _fields_ = [
        ("layers", C.c_int), ("batch", C.c_int), ("n_q_heads", C.c_int), ("n_kv_heads", C.c_int),
        ("head_dim", C.c_int), ("C", C.c_int), ("R", C.c_int), ("fusion", C.c_int), ("dtype", C.c_int),
        ("evict_interval", C.c_int), ("kernel", C.c_int), ("splits", C.c_int),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("norm_mode", C.c_int), ("full_layers", C.c_int),
        ("max_tokens", C.c_int), ("profile_mode", C.c_int),
        ("wait_limit_cycles", C.c_ulonglong),
    ]


class mkv_view(C.Structure):
    _fields_ = [
        ("K", C.c_void_p), ("V", C.c_void_p), ("pos", C.c_void_p), ("F", C.c_void_p), ("evicted_pos", C.c_void_p),
        ("ring_q", C.c_void_p), ("ring_c", C.c_void_p), ("count", C.c_int32), ("capacity", C.c_int32),
        ("next_pos", C.c_int64), ("group_stride", C.c_int32),
    ]


class MkvError(RuntimeError):
    def __init__(self, status: int, where: str, text: str = ""):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES[status] if 0 <= status < 7 else status} {text}".strip())


_lib = None


def lib() -> C.CDLL:
    """The loaded library.  Raises if it has not been built (``python -m paper_2503_00979_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2503_00979_b200.build` "
                              "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        vp, ip = C.c_void_p, C.c_int
        L.mkv_default_params.argtypes = [C.POINTER(mkv_params)]
        L.mkv_default_params.restype = None
        L.mkv_workspace_bytes.argtypes = [C.POINTER(mkv_params)]
        L.mkv_workspace_bytes.restype = C.c_size_t
        L.mkv_create.argtypes = [C.POINTER(vp), ip, ip, ip, ip, ip, ip, ip, ip]
        L.mkv_create_ex.argtypes = [C.POINTER(vp), C.POINTER(mkv_params)]
        L.mkv_destroy.argtypes = [vp]
        L.mkv_destroy.restype = None
        L.mkv_reset.argtypes = [vp]
        L.mkv_prefill.argtypes = [vp, vp, vp, vp, ip, vp]
        L.mkv_prefill_static.argtypes = [vp, vp, vp, vp, ip, vp]
        L.mkv_prefill_ragged.argtypes = [vp, vp, vp, vp, C.POINTER(C.c_int32), ip, vp]
        L.mkv_row_state.argtypes = [vp, ip, C.POINTER(C.c_int32), C.POINTER(C.c_int64)]
        L.mkv_decode_step.argtypes = [vp, vp, vp, vp, vp, vp]
        L.mkv_decode_step_layer.argtypes = [vp, ip, vp, vp, vp, vp, vp]
        L.mkv_decode_steps.argtypes = [vp, vp, vp, vp, vp, ip, vp]
        L.mkv_decode_step_host.argtypes = [vp, vp, vp, vp, vp, vp]
        L.mkv_cache_view.argtypes = [vp, ip, C.POINTER(mkv_view)]
        L.mkv_sync.argtypes = [vp, vp]
        L.mkv_last_error.argtypes = [vp]
        L.mkv_last_error.restype = C.c_char_p
        L.mkv_launch_count.argtypes = [vp]
        L.mkv_launch_count.restype = C.c_uint64
        L.mkv_kernel_name.argtypes = [vp]
        L.mkv_kernel_name.restype = C.c_char_p
        _lib = L
    return _lib


def _ptr(x) -> int:
    """Address of a torch tensor (device or host) or a raw integer address."""
    if isinstance(x, torch.Tensor):
        assert x.is_contiguous(), "tensors passed to the library must be contiguous"
        return x.data_ptr()
    return int(x) if x is not None else 0


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if isinstance(stream, torch.cuda.Stream) else int(stream)


# ---- one function per C entry point -------------------------------------------------------
def mkv_default_params() -> mkv_params:
    p = mkv_params()
    lib().mkv_default_params(C.byref(p))
    return p


def mkv_workspace_bytes(p: mkv_params) -> int:
    return lib().mkv_workspace_bytes(C.byref(p))


def mkv_create(layers, batch, n_q_heads, n_kv_heads, head_dim, C_, R, fusion) -> tuple[int, int]:
    h = C.c_void_p()
    st = lib().mkv_create(C.byref(h), layers, batch, n_q_heads, n_kv_heads, head_dim, C_, R, int(fusion))
    return st, h.value


def mkv_create_ex(p: mkv_params) -> tuple[int, int]:
    h = C.c_void_p()
    st = lib().mkv_create_ex(C.byref(h), C.byref(p))
    return st, h.value


def mkv_destroy(ctx) -> None:
    lib().mkv_destroy(ctx)


def mkv_reset(ctx) -> int:
    return lib().mkv_reset(ctx)


def mkv_prefill(ctx, k, v, q_window, prompt_len, stream=None) -> int:
    return lib().mkv_prefill(ctx, _ptr(k), _ptr(v), _ptr(q_window), prompt_len, _stream(stream))


def mkv_prefill_ragged(ctx, k, v, q_window, prompt_lens, padded_len, stream=None) -> int:
    """Prompt phase of a batch whose rows have different prompt lengths (tensors padded to padded_len)."""
    lens = (C.c_int32 * len(prompt_lens))(*[int(x) for x in prompt_lens])
    return lib().mkv_prefill_ragged(ctx, _ptr(k), _ptr(v), _ptr(q_window), lens, padded_len, _stream(stream))


def mkv_row_state(ctx, layer, batch):
    """(status, counts, next positions) of the batch rows as `layer` holds them."""
    cnt, nxt = (C.c_int32 * batch)(), (C.c_int64 * batch)()
    st = lib().mkv_row_state(ctx, layer, cnt, nxt)
    return st, list(cnt), list(nxt)


def mkv_prefill_static(ctx, k, v, q_window, prompt_len, stream=None) -> int:
    """mkv_prefill without any device allocation (scratch in the library's fixed 16 MiB array)."""
    return lib().mkv_prefill_static(ctx, _ptr(k), _ptr(v), _ptr(q_window), prompt_len, _stream(stream))


def mkv_decode_step(ctx, q, k_new, v_new, out, stream=None) -> int:
    return lib().mkv_decode_step(ctx, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _stream(stream))


def mkv_decode_step_layer(ctx, layer, q, k_new, v_new, out, stream=None) -> int:
    return lib().mkv_decode_step_layer(ctx, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _stream(stream))


def mkv_decode_steps(ctx, q, k_new, v_new, out, n_steps, stream=None) -> int:
    return lib().mkv_decode_steps(ctx, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), n_steps, _stream(stream))


def mkv_decode_step_host(ctx, q_host, k_new_host, v_new_host, out_host, stream=None) -> int:
    return lib().mkv_decode_step_host(ctx, _ptr(q_host), _ptr(k_new_host), _ptr(v_new_host), _ptr(out_host),
                                      _stream(stream))


def mkv_cache_view(ctx, layer: int) -> tuple[int, mkv_view]:
    v = mkv_view()
    st = lib().mkv_cache_view(ctx, layer, C.byref(v))
    return st, v


def mkv_sync(ctx, stream=None) -> int:
    return lib().mkv_sync(ctx, _stream(stream))


def mkv_last_error(ctx) -> str:
    return lib().mkv_last_error(ctx).decode()


def mkv_launch_count(ctx) -> int:
    return lib().mkv_launch_count(ctx)


def mkv_kernel_name(ctx) -> str:
    return lib().mkv_kernel_name(ctx).decode()


# ---- convenience holder ---------------------------------------------------------------------
def _from_ptr(ptr: int, shape, dtype: torch.dtype, device) -> torch.Tensor:
    """A torch view of library-owned device memory (no copy) through the CUDA array interface."""
    n = 1
    for s in shape:
        n *= s
    itemsize = torch.empty((), dtype=dtype).element_size()
    typestr = {torch.float32: "<f4", torch.int32: "<i4", torch.bfloat16: "<i2"}[dtype]

    class _Holder:
        __cuda_array_interface__ = {"shape": (n,), "typestr": typestr, "data": (ptr, False), "version": 2}

    t = torch.as_tensor(_Holder(), device=device)
    if dtype == torch.bfloat16:
        t = t.view(torch.bfloat16)
    assert t.element_size() == itemsize
    return t.view(*shape)


class MorphKV:
    """A context whose workspace is a torch tensor.  Methods mirror the C calls and raise on error."""

    def __init__(self, layers, batch, n_q_heads, n_kv_heads, head_dim, C_, R, fusion="sum", dtype="bf16",
                 evict_interval=1, kernel="auto", splits=0, device="cuda:0", wait_limit_cycles=0,
                 full_layers=0, max_tokens=0, norm="frozen", profile="recompute"):
        self.device = torch.device(device)
        p = mkv_default_params()
        p.layers, p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim = layers, batch, n_q_heads, n_kv_heads, head_dim
        p.C, p.R = C_, R
        p.fusion = FUSION[fusion] if isinstance(fusion, str) else int(fusion)
        p.dtype = DTYPE[dtype] if isinstance(dtype, str) else int(dtype)
        p.evict_interval, p.kernel, p.splits = evict_interval, KERNEL[kernel], splits
        p.wait_limit_cycles = wait_limit_cycles
        p.full_layers, p.max_tokens = full_layers, max_tokens
        p.norm_mode = NORM[norm]
        p.profile_mode = PROFILE[profile]
        self.torch_dtype = torch.float32 if p.dtype == 1 else torch.bfloat16
        self.shape = dict(L=layers, B=batch, Hq=n_q_heads, Hkv=n_kv_heads, d=head_dim, C=C_, R=R,
                          G=n_q_heads // max(1, n_kv_heads))
        nbytes = mkv_workspace_bytes(p)
        self.ctx = None
        if nbytes == 0:
            st, _ = mkv_create_ex(p)          # let the library say why
            raise MkvError(st if st else INVALID_ARG, "mkv_create_ex")
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = (self.workspace.data_ptr() + 255) & ~255
            p.workspace, p.workspace_bytes = base, nbytes
            st, h = mkv_create_ex(p)
        if st != OK:
            raise MkvError(st, "mkv_create_ex")
        self.ctx = h
        self.params = p

    def close(self):
        if getattr(self, "ctx", None):
            mkv_destroy(self.ctx)
            self.ctx = None

    __del__ = close

    def _check(self, st, where):
        if st != OK:
            raise MkvError(st, where, mkv_last_error(self.ctx))

    def reset(self):
        self._check(mkv_reset(self.ctx), "mkv_reset")

    def prefill(self, k, v, q_window, stream=None):
        self._check(mkv_prefill(self.ctx, k, v, q_window, k.shape[-2], stream), "mkv_prefill")

    def prefill_ragged(self, k, v, q_window, prompt_lens, stream=None):
        """Prompt phase with one prompt length per batch row; k, v are padded to k.shape[-2] tokens."""
        if len(prompt_lens) != self.shape["B"]:
            raise ValueError("one prompt length per batch row")
        self._check(mkv_prefill_ragged(self.ctx, k, v, q_window, prompt_lens, k.shape[-2], stream), "mkv_prefill_ragged")

    def row_state(self, layer: int):
        """(cached tokens, next position) of every batch row in `layer`."""
        st, cnt, nxt = mkv_row_state(self.ctx, layer, self.shape["B"])
        self._check(st, "mkv_row_state")
        return cnt, nxt

    def prefill_static(self, k, v, q_window, stream=None):
        """Prompt phase for hosts that cannot allocate device memory; see mkv_prefill_static in mkv.h."""
        self._check(mkv_prefill_static(self.ctx, k, v, q_window, k.shape[-2], stream), "mkv_prefill_static")

    def decode_step(self, q, k_new, v_new, out=None, stream=None):
        if out is None:
            out = torch.empty_like(q)
        self._check(mkv_decode_step(self.ctx, q, k_new, v_new, out, stream), "mkv_decode_step")
        return out

    def decode_step_layer(self, layer, q, k_new, v_new, out=None, stream=None):
        if out is None:
            out = torch.empty_like(q)
        self._check(mkv_decode_step_layer(self.ctx, layer, q, k_new, v_new, out, stream), "mkv_decode_step_layer")
        return out

    def decode_steps(self, q, k_new, v_new, out=None, stream=None):
        if out is None:
            out = torch.empty_like(q)
        self._check(mkv_decode_steps(self.ctx, q, k_new, v_new, out, q.shape[0], stream), "mkv_decode_steps")
        return out

    def decode_step_host(self, q_host, k_new_host, v_new_host, out_host, stream=None):
        self._check(mkv_decode_step_host(self.ctx, q_host, k_new_host, v_new_host, out_host, stream),
                    "mkv_decode_step_host")
        return out_host

    def sync(self, stream=None):
        self._check(mkv_sync(self.ctx, stream), "mkv_sync")

    def view(self, layer: int) -> dict:
        """Torch views (no copies) of one layer of the cache; synchronise before reading."""
        st, v = mkv_cache_view(self.ctx, layer)
        self._check(st, "mkv_cache_view")
        s = self.shape
        B, H, cap, d, R, G = s["B"], s["Hkv"], v.capacity, s["d"], s["R"], v.group_stride
        dev = self.device
        return dict(
            K=_from_ptr(v.K, (B, H, cap, d), self.torch_dtype, dev),
            V=_from_ptr(v.V, (B, H, cap, d), self.torch_dtype, dev),
            pos=_from_ptr(v.pos, (B, H, cap), torch.int32, dev),
            F=_from_ptr(v.F, (B, H, cap), torch.float32, dev),
            evicted_pos=_from_ptr(v.evicted_pos, (B, H), torch.int32, dev),
            ring_q=_from_ptr(v.ring_q, (B, H, R, G, d), self.torch_dtype, dev),
            ring_c=_from_ptr(v.ring_c, (B, H, R, G), torch.float32, dev),
            count=v.count, capacity=cap, next_pos=v.next_pos,
        )

    @property
    def launch_count(self) -> int:
        return mkv_launch_count(self.ctx)

    @property
    def kernel_name(self) -> str:
        return mkv_kernel_name(self.ctx)
