"""Thin ctypes binding of the C ABI declared in include/amph.h.

Only argument marshalling happens here: every step of the decoding path runs in the CUDA
kernels of libamph.so.  PyTorch is used to allocate device memory and to provide the stream.
There is no fallback: if the shared library is missing, importing `lib()` raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
AMPH_MAX_HEADS_K = 8
AMPH_MAX_NODES = 128
AMPH_TOPK_STRIDE = 16
AMPH_DTYPE_F32, AMPH_DTYPE_BF16 = 0, 1
AMPH_FLAG_NO_TENSOR_CORE, AMPH_FLAG_NO_GRAPH, AMPH_FLAG_SEPARATE_ROPE = 1, 2, 4
AMPH_FLAG_SEPARATE_MERGE, AMPH_FLAG_SEPARATE_SWIGLU, AMPH_FLAG_MMA_SYNC_ATTENTION, AMPH_FLAG_NO_SAMPLED_TOKEN = 8, 16, 32, 64
AMPH_FLAG_CHUNKED_PREFILL, AMPH_FLAG_NO_SIDE_PREFETCH = 128, 256
STATUS = {0: "AMPH_OK", 1: "AMPH_ERR_INVALID_ARG", 2: "AMPH_ERR_SHAPE", 3: "AMPH_ERR_STATE",
          4: "AMPH_ERR_CAPACITY", 5: "AMPH_ERR_WORKSPACE", 6: "AMPH_ERR_MISSING_WEIGHT",
          7: "AMPH_ERR_CUDA", 8: "AMPH_ERR_TIMEOUT"}
EXPORTS = ["amph_workspace_bytes", "amph_init", "amph_load_weights", "amph_prefill", "amph_prefill_seq", "amph_get_state_seq", "amph_draft",
           "amph_verify_tree", "amph_accept", "amph_step", "amph_get_tensor", "amph_set_tensor",
           "amph_get_state", "amph_set_state", "amph_selftest_wait_timeout", "amph_profile_begin", "amph_profile_end", "amph_profile_breakdown", "amph_project", "amph_project_noalloc",
           "amph_reset", "amph_destroy", "amph_last_error"]


class amph_config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("head_dim", C.c_int32), ("d_ffn", C.c_int32), ("vocab", C.c_int32),
                ("rms_eps", C.c_float), ("rope_theta", C.c_float),
                ("weight_dtype", C.c_int32), ("kv_dtype", C.c_int32), ("max_ctx", C.c_int32),
                ("max_batch", C.c_int32), ("K", C.c_int32), ("n_sal", C.c_int32),
                ("aeb_layers", C.c_int32), ("topk", C.c_int32 * AMPH_MAX_HEADS_K), ("flags", C.c_int32),
                ("lm_rank", C.c_int32), ("temperature", C.c_float), ("seed_lo", C.c_uint32), ("seed_hi", C.c_uint32)]


class amph_tree(C.Structure):
    _fields_ = [("n_nodes", C.c_int32), ("parent", C.POINTER(C.c_int16)),
                ("depth", C.POINTER(C.c_uint8)), ("rank", C.POINTER(C.c_uint8))]


class amph_tensor(C.Structure):
    _fields_ = [("name", C.c_char_p), ("dev_ptr", C.c_void_p), ("dtype", C.c_int32),
                ("ndim", C.c_int32), ("shape", C.c_int64 * 4)]


class AmphError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS.get(status, status)}: {message}")
        self.status = status


def library_path() -> str:
    return os.path.join(_HERE, "libamph.so")


_lib = None


def lib() -> C.CDLL:
    """Loads libamph.so (built by paper_2406_13170_b200/build.py).  Raises if it is missing."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise FileNotFoundError(f"{path} is missing: run `python -m paper_2406_13170_b200.build` "
                                    "(there is no CPU or PyTorch fallback for the decoding path)")
        L = C.CDLL(path)
        vp, i32p, f32p = C.c_void_p, C.c_void_p, C.c_void_p
        L.amph_workspace_bytes.argtypes = [C.POINTER(amph_config), C.POINTER(amph_tree),
                                           C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
        L.amph_init.argtypes = [C.POINTER(amph_config), C.POINTER(amph_tree), vp, C.c_size_t, vp,
                                C.c_size_t, vp, C.POINTER(vp)]
        L.amph_load_weights.argtypes = [vp, C.POINTER(amph_tensor), C.c_int32]
        L.amph_prefill.argtypes = [vp, C.POINTER(C.c_int32), C.c_int32, C.POINTER(C.c_int32)]
        L.amph_prefill_seq.argtypes = [vp, C.c_int32, C.POINTER(C.c_int32), C.c_int32, C.POINTER(C.c_int32)]
        L.amph_get_state_seq.argtypes = [vp, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.amph_draft.argtypes = [vp, i32p, f32p]
        L.amph_verify_tree.argtypes = [vp, i32p, i32p]
        L.amph_accept.argtypes = [vp, i32p, i32p, i32p, i32p]
        L.amph_step.argtypes = [vp, i32p, i32p]
        L.amph_get_tensor.argtypes = [vp, C.c_char_p, vp, C.c_size_t]
        L.amph_set_tensor.argtypes = [vp, C.c_char_p, vp, C.c_size_t]
        L.amph_get_state.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.amph_set_state.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, vp, C.POINTER(C.c_int32)]
        L.amph_selftest_wait_timeout.argtypes = [vp, C.c_int32, C.POINTER(vp), C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                                 vp, vp, C.c_size_t, vp, C.c_int32]
        L.amph_profile_begin.argtypes = [vp]
        L.amph_profile_end.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        L.amph_profile_breakdown.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
        L.amph_project.argtypes = [vp, C.c_int32, C.POINTER(vp), C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                   C.c_int32, C.c_int32, vp, vp, C.c_size_t, vp]
        L.amph_project_noalloc.argtypes = [vp, C.c_int32, C.POINTER(vp), C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                           C.c_int32, C.c_int32, vp, vp, vp, C.c_char_p, C.c_size_t]
        L.amph_reset.argtypes = [vp]
        L.amph_destroy.argtypes = [vp]
        L.amph_destroy.restype = None
        L.amph_last_error.argtypes = [vp]
        L.amph_last_error.restype = C.c_char_p
        for name in EXPORTS:
            if name not in ("amph_destroy", "amph_last_error"):
                getattr(L, name).restype = C.c_int32
        _lib = L
    return _lib


def make_config(shape, max_ctx: Optional[int] = None, flags: int = 0, max_batch: int = 1, temperature: float = 0.0,
                seed: int = 0) -> amph_config:
    """amph_config from an object with the fields of inputs.configs.ModelShape."""
    c = amph_config()
    c.n_layers, c.d_model, c.n_heads, c.head_dim = shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim
    c.d_ffn, c.vocab, c.rms_eps, c.rope_theta = shape.d_ffn, shape.vocab, shape.rms_eps, shape.rope_theta
    dt = AMPH_DTYPE_F32 if shape.dtype == "fp32" else AMPH_DTYPE_BF16
    c.weight_dtype = c.kv_dtype = dt
    c.max_ctx = int(max_ctx or shape.ctx_capacity)
    c.max_batch = int(max_batch)
    c.K, c.n_sal, c.aeb_layers = shape.K, shape.n_sal, shape.aeb_layers
    c.lm_rank = getattr(shape, "lm_rank", 0)
    for k in range(shape.K):
        c.topk[k] = shape.topk[k]
    c.flags = flags | (0 if getattr(shape, "use_sampled_token", True) else AMPH_FLAG_NO_SAMPLED_TOKEN)
    c.temperature = float(temperature)
    c.seed_lo, c.seed_hi = int(seed) & 0xFFFFFFFF, (int(seed) >> 32) & 0xFFFFFFFF
    return c


class _TreeHolder:
    """amph_tree plus the host arrays it points to."""

    def __init__(self, parent: Sequence[int], depth: Sequence[int], rank: Sequence[int]):
        n = len(parent)
        self.parent = (C.c_int16 * n)(*parent)
        self.depth = (C.c_uint8 * n)(*depth)
        self.rank = (C.c_uint8 * n)(*rank)
        self.c = amph_tree(n, self.parent, self.depth, self.rank)


def make_tree(topo) -> _TreeHolder:
    return _TreeHolder(topo.parent, topo.depth, topo.rank)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


class Amphista:
    """One decoding context.  Owns the device regions (torch tensors) the C library borrows."""

    def __init__(self, shape, topo, weights: Dict[str, torch.Tensor], device="cuda:0",
                 max_ctx: Optional[int] = None, flags: int = 0, stream: Optional[torch.cuda.Stream] = None,
                 max_batch: int = 1, temperature: float = 0.0, seed: int = 0):
        self.L = lib()
        self.shape, self.topo = shape, topo
        self.device = torch.device(device)
        self.B = int(max_batch)
        self.cfg = make_config(shape, max_ctx, flags, max_batch, temperature, seed)
        self.tree = make_tree(topo)
        kvb, wsb = C.c_size_t(), C.c_size_t()
        self._check(self.L.amph_workspace_bytes(C.byref(self.cfg), C.byref(self.tree.c), C.byref(kvb), C.byref(wsb)), None)
        with torch.cuda.device(self.device):
            self.kv = torch.empty(kvb.value, dtype=torch.uint8, device=self.device)
            self.ws = torch.empty(wsb.value, dtype=torch.uint8, device=self.device)
            # a stream of its own: the legacy default stream cannot be captured into a CUDA graph
            self.stream = stream or torch.cuda.Stream(self.device)
            self.stream.wait_stream(torch.cuda.current_stream(self.device))
            self.ctx = C.c_void_p()
            self._check(self.L.amph_init(C.byref(self.cfg), C.byref(self.tree.c), _ptr(self.kv), kvb.value,
                                         _ptr(self.ws), wsb.value, C.c_void_p(self.stream.cuda_stream),
                                         C.byref(self.ctx)), None)
        self.weights = weights            # keeps the tensors alive
        self.load_weights(weights)
        N, K = topo.n_nodes, shape.K
        self.out_tokens = torch.empty(self.B, K + 1, dtype=torch.int32, device=self.device)
        self.out_n = torch.empty(self.B, dtype=torch.int32, device=self.device)

    def _after_torch(self) -> None:
        """Orders the library's stream after work torch has queued on its current stream (inputs)."""
        self.stream.wait_stream(torch.cuda.current_stream(self.device))

    def synchronize(self) -> None:
        self.stream.synchronize()

    def _check(self, status: int, ctx) -> None:
        if status != 0:
            raise AmphError(status, self.L.amph_last_error(ctx).decode())

    def load_weights(self, weights: Dict[str, torch.Tensor]) -> None:
        arr = (amph_tensor * len(weights))()
        keep = []
        for i, (name, t) in enumerate(weights.items()):
            assert t.is_cuda and t.is_contiguous(), name
            b = name.encode()
            keep.append(b)
            arr[i].name = b
            arr[i].dev_ptr = t.data_ptr()
            arr[i].dtype = AMPH_DTYPE_F32 if t.dtype == torch.float32 else AMPH_DTYPE_BF16
            arr[i].ndim = t.dim()
            for j, s in enumerate(t.shape):
                arr[i].shape[j] = s
        self._after_torch()
        self._check(self.L.amph_load_weights(self.ctx, arr, len(weights)), self.ctx)

    def prefill(self, prompt: Sequence[int], seq: int = 0) -> int:
        n = len(prompt)
        ids = (C.c_int32 * n)(*[int(t) for t in prompt])
        root = C.c_int32()
        with torch.cuda.device(self.device):
            self._check(self.L.amph_prefill_seq(self.ctx, int(seq), ids, n, C.byref(root)), self.ctx)
        return root.value

    def draft(self, out_ids: Optional[torch.Tensor] = None, out_vals: Optional[torch.Tensor] = None) -> None:
        with torch.cuda.device(self.device):
            self._check(self.L.amph_draft(self.ctx, _ptr(out_ids), _ptr(out_vals)), self.ctx)

    def verify_tree(self, tree_tokens: Optional[torch.Tensor] = None, out_argmax: Optional[torch.Tensor] = None) -> None:
        self._after_torch()
        with torch.cuda.device(self.device):
            self._check(self.L.amph_verify_tree(self.ctx, _ptr(tree_tokens), _ptr(out_argmax)), self.ctx)

    def accept(self, out_tokens=None, out_n=None, out_path=None, out_next_root=None) -> None:
        with torch.cuda.device(self.device):
            self._check(self.L.amph_accept(self.ctx, _ptr(out_tokens), _ptr(out_n), _ptr(out_path),
                                           _ptr(out_next_root)), self.ctx)

    def step(self, out_tokens: Optional[torch.Tensor] = None, out_n: Optional[torch.Tensor] = None) -> None:
        with torch.cuda.device(self.device):
            self._check(self.L.amph_step(self.ctx, _ptr(out_tokens), _ptr(out_n)), self.ctx)

    def get_tensor(self, name: str, shape, dtype=torch.float32) -> torch.Tensor:
        out = torch.empty(shape, dtype=dtype, device=self.device)
        with torch.cuda.device(self.device):
            self._check(self.L.amph_get_tensor(self.ctx, name.encode(), _ptr(out), out.numel() * out.element_size()),
                        self.ctx)
        self.stream.synchronize()
        return out

    def set_tensor(self, name: str, src: torch.Tensor) -> None:
        self._after_torch()
        with torch.cuda.device(self.device):
            self._check(self.L.amph_set_tensor(self.ctx, name.encode(), _ptr(src), src.numel() * src.element_size()),
                        self.ctx)

    def get_state(self, seq: int = 0):
        a, b, c = C.c_int32(), C.c_int32(), C.c_int32()
        with torch.cuda.device(self.device):
            self._check(self.L.amph_get_state_seq(self.ctx, int(seq), C.byref(a), C.byref(b), C.byref(c)), self.ctx)
        return a.value, b.value, c.value

    def set_state(self, ctx_len: int, root: int, pend_hidden: torch.Tensor, pend_next: Sequence[int]) -> None:
        """amph_set_state: pend_hidden f32 [n_pending, d] (cpu or cuda), pend_next the token after each pending row."""
        n = len(pend_next)
        h = pend_hidden.to(torch.float32).contiguous()
        assert h.shape == (n, self.shape.d_model)
        ids = (C.c_int32 * n)(*[int(t) for t in pend_next])
        self._after_torch()
        with torch.cuda.device(self.device):
            self._check(self.L.amph_set_state(self.ctx, int(ctx_len), int(root), n, _ptr(h), ids), self.ctx)
            self.stream.synchronize()                 # h may be a temporary

    def profile_begin(self) -> None:
        self._check(self.L.amph_profile_begin(self.ctx), self.ctx)

    def profile_end(self):
        ms, n, by = C.c_double(), C.c_int64(), C.c_int64()
        with torch.cuda.device(self.device):
            self._check(self.L.amph_profile_end(self.ctx, C.byref(ms), C.byref(n), C.byref(by)), self.ctx)
        return ms.value, n.value, by.value

    PROF_NAMES = ["projection", "norm", "rope_kv", "attention", "swiglu", "select", "accept", "other"]

    def profile_breakdown(self):
        ms = (C.c_double * 8)()
        n = (C.c_int64 * 8)()
        self._check(self.L.amph_profile_breakdown(self.ctx, ms, n), self.ctx)
        return {k: (ms[i], n[i]) for i, k in enumerate(self.PROF_NAMES)}

    def reset(self) -> None:
        self._check(self.L.amph_reset(self.ctx), self.ctx)

    def close(self) -> None:
        if getattr(self, "ctx", None) and self.ctx.value:
            torch.cuda.synchronize(self.device)
            self.L.amph_destroy(self.ctx)
            self.ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def project(x: torch.Tensor, ws: Sequence[torch.Tensor], rows: int, use_tensor_core: bool) -> torch.Tensor:
    """amph_project: y[r][s*out + o] = sum_k x[r][k] * ws[s][o][k] for the first `rows` rows of x."""
    L = lib()
    n_seg = len(ws)
    out, in_ = ws[0].shape
    dev = x.device
    y = torch.empty(rows, n_seg * out, dtype=torch.float32, device=dev)
    scratch = torch.empty(256 + 16 * 128 * n_seg * out * 4, dtype=torch.uint8, device=dev)
    arr = (C.c_void_p * n_seg)(*[w.data_ptr() for w in ws])
    dt = AMPH_DTYPE_F32 if x.dtype == torch.float32 else AMPH_DTYPE_BF16
    with torch.cuda.device(dev):
        rc = L.amph_project(_ptr(x), x.shape[0], arr, n_seg, out, in_, rows, dt, int(use_tensor_core), _ptr(y),
                            _ptr(scratch), scratch.numel(), C.c_void_p(torch.cuda.current_stream(dev).cuda_stream))
        if rc != 0:
            raise AmphError(rc, L.amph_last_error(None).decode())
        torch.cuda.synchronize(dev)
    err = int(scratch[:4].view(torch.int32)[0])
    if err:
        raise AmphError(err, "a bounded device-side wait gave up")
    return y


def selftest_wait_timeout(x: torch.Tensor, ws: Sequence[torch.Tensor], rows: int, limit_us: int = 1000):
    """amph_selftest_wait_timeout: returns (status word read back from the scratch, y)."""
    L = lib()
    n_seg = len(ws)
    out, in_ = ws[0].shape
    dev = x.device
    y = torch.full((rows, n_seg * out), float("nan"), dtype=torch.float32, device=dev)
    scratch = torch.zeros(256 + 16 * 128 * n_seg * out * 4, dtype=torch.uint8, device=dev)
    arr = (C.c_void_p * n_seg)(*[w.data_ptr() for w in ws])
    with torch.cuda.device(dev):
        rc = L.amph_selftest_wait_timeout(_ptr(x), x.shape[0], arr, n_seg, out, in_, rows, _ptr(y), _ptr(scratch),
                                          scratch.numel(), C.c_void_p(torch.cuda.current_stream(dev).cuda_stream), limit_us)
        if rc != 0:
            raise AmphError(rc, L.amph_last_error(None).decode())
        torch.cuda.synchronize(dev)
    return int(scratch[:4].view(torch.int32)[0]), y


def project_noalloc(x: torch.Tensor, ws: Sequence[torch.Tensor], rows: int, use_tensor_core: bool,
                    y: torch.Tensor, status: Optional[torch.Tensor] = None) -> None:
    """amph_project_noalloc: like `project`, for callers that cannot allocate device memory when they
    call (all free memory already belongs to someone else's pool, or an allocation's hidden
    synchronisation is not acceptable).  The split-K scratch is a fixed array inside the library, so the
    caller passes only inputs and the preallocated outputs `y` (fp32 [rows, n_seg*out]) and, optionally,
    `status` (int32 [1]).  Nothing is allocated here either: no torch tensor is created.
    Calls share the built-in scratch: do not let two of them overlap on the GPU."""
    L = lib()
    n_seg = len(ws)
    out, in_ = ws[0].shape
    dev = x.device
    arr = (C.c_void_p * n_seg)(*[w.data_ptr() for w in ws])
    dt = AMPH_DTYPE_F32 if x.dtype == torch.float32 else AMPH_DTYPE_BF16
    msg = C.create_string_buffer(512)
    with torch.cuda.device(dev):
        rc = L.amph_project_noalloc(_ptr(x), x.shape[0], arr, n_seg, out, in_, rows, dt, int(use_tensor_core),
                                    _ptr(y), _ptr(status), C.c_void_p(torch.cuda.current_stream(dev).cuda_stream),
                                    msg, len(msg))
    if rc != 0:
        raise AmphError(rc, msg.value.decode())
