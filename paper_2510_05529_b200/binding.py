"""ctypes binding of libh1b.so: the same entry points as include/h1b.h.

This module only marshals arguments. Every step of the path (sketching,
quantisation, scores, softmax, weighted sum) runs in the CUDA library. PyTorch
is used for device memory and streams. There is no CPU fallback: a missing or
unloadable library raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

from .build import LIB_PATH, build_library, is_stale

H1B_OK = 0
ERRORS = {
    -1: "H1B_ERR_INVALID_ARG", -2: "H1B_ERR_NULL", -3: "H1B_ERR_UNSUPPORTED", -4: "H1B_ERR_CAPACITY",
    -5: "H1B_ERR_WORKSPACE", -6: "H1B_ERR_CUDA", -7: "H1B_ERR_TIMEOUT", -8: "H1B_ERR_BOUNDS",
}


class H1BError(RuntimeError):
    def __init__(self, code: int, text: str = ""):
        self.code = code
        super().__init__("%s (%d)%s" % (ERRORS.get(code, "H1B_ERR_?"), code, ": " + text if text else ""))


class h1b_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("n_layers", "n_q_heads", "n_kv_heads", "head_dim", "sketch_bits", "group_size",
                 "max_batch", "max_seq", "device")] + [("flags", ctypes.c_uint32), ("page_tokens", ctypes.c_int32),
                                                       ("n_pages", ctypes.c_int32)]


_lib = None


def load_library(rebuild: bool = True) -> ctypes.CDLL:
    """Load libh1b.so (building it with nvcc first when it is missing or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    path = os.environ.get("H1B_LIBRARY_PATH")          # a prebuilt library elsewhere; default: the in-tree one
    if not path:
        path = LIB_PATH
        if rebuild and is_stale():
            build_library()
    if not os.path.exists(path):
        raise RuntimeError("%s is missing and could not be built; there is no fallback path" % path)
    lib = ctypes.CDLL(path)
    vp, cp = ctypes.c_void_p, ctypes.POINTER(h1b_config)
    i32p = ctypes.POINTER(ctypes.c_int32)
    sig = {
        "h1b_entry_bytes": (ctypes.c_size_t, [cp]),
        "h1b_cache_bytes": (ctypes.c_size_t, [cp]),
        "h1b_init_projection": (ctypes.c_int, [cp, ctypes.c_uint64, vp, vp, ctypes.c_size_t, vp,
                                               ctypes.POINTER(vp)]),
        "h1b_append_kv": (ctypes.c_int, [vp, ctypes.c_int, ctypes.c_int, vp, vp, i32p, ctypes.c_int,
                                         ctypes.c_int, vp]),
        "h1b_decode_attention": (ctypes.c_int, [vp, ctypes.c_int, ctypes.c_int, vp, ctypes.c_float, vp,
                                                ctypes.c_int, vp]),
        "h1b_decode_attention_multi": (ctypes.c_int, [vp, ctypes.c_int, ctypes.c_int, vp, ctypes.c_int, ctypes.c_float,
                                                      vp, ctypes.c_int, vp]),
        "h1b_prefill_attention": (ctypes.c_int, [vp, ctypes.c_int, ctypes.c_int, vp, ctypes.c_int, ctypes.c_float,
                                                 vp, ctypes.c_int, vp]),
        "h1b_decode_attention_static": (ctypes.c_int, [vp, ctypes.c_int, ctypes.c_int, vp, ctypes.c_float, vp,
                                                       ctypes.c_int, vp]),
        "h1b_decode_step": (ctypes.c_int, [vp, vp, vp, vp, ctypes.c_float, vp, ctypes.c_int, vp]),
        "h1b_decode_step_layers": (ctypes.c_int, [vp, ctypes.c_int, ctypes.c_int, vp, vp, vp, ctypes.c_float, vp,
                                                  ctypes.c_int, vp]),
        "h1b_sync_lengths": (ctypes.c_int, [vp, vp]),
        "h1b_set_block_table": (ctypes.c_int, [vp, ctypes.c_int, i32p, ctypes.c_int, vp]),
        "h1b_set_rope_table": (ctypes.c_int, [vp, vp, ctypes.c_int, vp]),
        "h1b_decode_step_host": (ctypes.c_int, [vp, vp, vp, vp, ctypes.c_float, vp, ctypes.c_int, vp]),
        "h1b_free": (ctypes.c_int, [vp]),
        "h1b_get_projection": (ctypes.c_int, [vp, ctypes.c_int, vp]),
        "h1b_get_lengths": (ctypes.c_int, [vp, ctypes.c_int, vp]),
        "h1b_reset": (ctypes.c_int, [vp, ctypes.c_int]),
        "h1b_truncate": (ctypes.c_int, [vp, ctypes.c_int, ctypes.c_int]),
        "h1b_truncate_async": (ctypes.c_int, [vp, ctypes.c_int, ctypes.c_int, vp]),
        "h1b_export_cache": (ctypes.c_int, [vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                            ctypes.c_int, vp, vp, vp, vp]),
        "h1b_export_values": (ctypes.c_int, [vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                             ctypes.c_int, vp]),
        "h1b_debug_scores": (ctypes.c_int, [vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp, vp, vp]),
        "h1b_debug_partials": (ctypes.c_int, [vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, i32p, vp, vp,
                                              ctypes.c_int]),
        "h1b_debug_wait_timeout": (ctypes.c_int, [vp, ctypes.c_uint64, vp]),
        "h1b_debug_prompt_scores": (ctypes.c_int, [vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp, ctypes.c_int]),
        "h1b_debug_prompt_route": (ctypes.c_int, [vp, ctypes.c_int]),
        "h1b_debug_prompt_stall": (ctypes.c_int, [vp, ctypes.c_uint64]),
        "h1b_bounds_checked": (ctypes.c_int, []),
        "h1b_debug_bounds_probe": (ctypes.c_int, [vp, vp]),
        "h1b_set_splits": (ctypes.c_int, [vp, ctypes.c_int]),
        "h1b_poll_status": (ctypes.c_int, [vp]),
        "h1b_set_profiling": (ctypes.c_int, [vp, ctypes.c_int]),
        "h1b_read_profile": (ctypes.c_int, [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int64)]),
        "h1b_launch_count": (ctypes.c_int64, [vp]),
        "h1b_last_error": (ctypes.c_char_p, [vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


H1B_FLAG_FP16_VALUES = 1      # h1b_config.flags: values stay fp16 (the 1-bit-keys-only configuration)
H1B_FLAG_ROPE = 2             # keys and queries are rotated (rotary position embedding) before they are sketched


def make_config(n_layers, n_q_heads, n_kv_heads, head_dim=128, sketch_bits=128, group_size=32,
                max_batch=1, max_seq=8192, device=0, fp16_values=False, page_tokens=0, n_pages=0,
                rope=False) -> h1b_config:
    """page_tokens > 0: a paged cache with n_pages pages of that many tokens in each layer's pool."""
    flags = (H1B_FLAG_FP16_VALUES if fp16_values else 0) | (H1B_FLAG_ROPE if rope else 0)
    return h1b_config(n_layers, n_q_heads, n_kv_heads, head_dim, sketch_bits, group_size,
                      max_batch, max_seq, device, flags, page_tokens, n_pages)


def h1b_bounds_checked() -> bool:
    """Whether the loaded library carries the kernels' index checks (built with H1B_DEBUG_BOUNDS=1)."""
    return bool(load_library().h1b_bounds_checked())


def h1b_entry_bytes(cfg: h1b_config) -> int:
    return int(load_library().h1b_entry_bytes(ctypes.byref(cfg)))


def h1b_cache_bytes(cfg: h1b_config) -> int:
    return int(load_library().h1b_cache_bytes(ctypes.byref(cfg)))


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _dev_ptr(t: torch.Tensor, dtype, what: str) -> int:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError("%s must be a contiguous CUDA tensor of dtype %s" % (what, dtype))
    return t.data_ptr()


class H1BCache:
    """One library context over a torch-owned device workspace."""

    def __init__(self, cfg: h1b_config, seed: int = 0, Rt: np.ndarray | None = None, stream=None):
        self.lib = load_library()
        self.cfg = cfg
        nbytes = h1b_cache_bytes(cfg)
        if nbytes == 0:
            raise H1BError(-3, "invalid or unsupported configuration")
        self.device = torch.device("cuda", cfg.device)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = self.workspace.data_ptr()
        self._ws_ptr = (base + 255) // 256 * 256
        self.workspace_bytes = nbytes
        rt_ptr = None
        if Rt is not None:
            Rt = np.ascontiguousarray(Rt, dtype=np.float32)
            want = (cfg.n_layers, cfg.head_dim, cfg.sketch_bits)
            if Rt.shape != want:
                raise ValueError("Rt must have shape %s, got %s" % (want, Rt.shape))
            rt_ptr = Rt.ctypes.data
        handle = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            rc = self.lib.h1b_init_projection(ctypes.byref(cfg), seed, rt_ptr, self._ws_ptr, nbytes,
                                              _stream_ptr(stream), ctypes.byref(handle))
        if rc != H1B_OK:
            raise H1BError(rc, (self.lib.h1b_last_error(None) or b"").decode())
        self._h = handle

    # -- helpers ---------------------------------------------------------
    def _check(self, rc: int):
        if rc != H1B_OK:
            raise H1BError(rc, (self.lib.h1b_last_error(self._h) or b"").decode())

    def close(self):
        if getattr(self, "_h", None):
            self.lib.h1b_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the four calls of the path ----------------------------------------
    def h1b_append_kv(self, k: torch.Tensor, v: torch.Tensor, layer_begin: int = 0, n_new=None, stream=None):
        """k, v: fp16 CUDA [n_layers, B, Tn, Hkv, d]."""
        kp = _dev_ptr(k, torch.float16, "k")
        vp = _dev_ptr(v, torch.float16, "v")
        if k.shape != v.shape or k.dim() != 5 or k.shape[3] != self.cfg.n_kv_heads or k.shape[4] != self.cfg.head_dim:
            raise ValueError("k and v must be [n_layers, B, Tn, Hkv, d]")
        nl, B, Tn = int(k.shape[0]), int(k.shape[1]), int(k.shape[2])
        nn = None
        if n_new is not None:
            arr = np.ascontiguousarray(n_new, dtype=np.int32)
            if arr.shape != (B,):
                raise ValueError("n_new must have shape [B]")
            nn = arr.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
        self._check(self.lib.h1b_append_kv(self._h, layer_begin, nl, kp, vp, nn, B, Tn, _stream_ptr(stream)))

    def h1b_decode_attention(self, q: torch.Tensor, inv_tau: float, out: torch.Tensor | None = None,
                             layer_begin: int = 0, stream=None) -> torch.Tensor:
        """q: fp16 CUDA [n_layers, B, Hq, d] -> out fp32 [n_layers, B, Hq, d]."""
        qp = _dev_ptr(q, torch.float16, "q")
        if q.dim() != 4 or q.shape[2] != self.cfg.n_q_heads or q.shape[3] != self.cfg.head_dim:
            raise ValueError("q must be [n_layers, B, Hq, d]")
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
        op = _dev_ptr(out, torch.float32, "out")
        if out.shape != q.shape:
            raise ValueError("out must have q's shape")
        self._check(self.lib.h1b_decode_attention(self._h, layer_begin, int(q.shape[0]), qp, float(inv_tau), op,
                                                  int(q.shape[1]), _stream_ptr(stream)))
        return out

    def h1b_decode_attention_multi(self, q: torch.Tensor, inv_tau: float, out: torch.Tensor | None = None,
                                   layer_begin: int = 0, stream=None) -> torch.Tensor:
        """q: fp16 CUDA [n_layers, B, Tq, Hq, d], the sequences' last Tq cached tokens -> out fp32, same shape."""
        qp = _dev_ptr(q, torch.float16, "q")
        if q.dim() != 5 or q.shape[3] != self.cfg.n_q_heads or q.shape[4] != self.cfg.head_dim:
            raise ValueError("q must be [n_layers, B, Tq, Hq, d]")
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
        op = _dev_ptr(out, torch.float32, "out")
        self._check(self.lib.h1b_decode_attention_multi(self._h, layer_begin, int(q.shape[0]), qp, int(q.shape[2]),
                                                        float(inv_tau), op, int(q.shape[1]), _stream_ptr(stream)))
        return out

    def h1b_prefill_attention(self, q: torch.Tensor, inv_tau: float, out: torch.Tensor | None = None,
                              layer_begin: int = 0, stream=None) -> torch.Tensor:
        """q: fp16 CUDA [n_layers, B, Tn, Hq, d], the sequences' last Tn cached tokens (any Tn) -> out fp32, same shape."""
        qp = _dev_ptr(q, torch.float16, "q")
        if q.dim() != 5 or q.shape[3] != self.cfg.n_q_heads or q.shape[4] != self.cfg.head_dim:
            raise ValueError("q must be [n_layers, B, Tn, Hq, d]")
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
        op = _dev_ptr(out, torch.float32, "out")
        if out.shape != q.shape:
            raise ValueError("out must have q's shape")
        self._check(self.lib.h1b_prefill_attention(self._h, layer_begin, int(q.shape[0]), qp, int(q.shape[2]),
                                                   float(inv_tau), op, int(q.shape[1]), _stream_ptr(stream)))
        return out

    def h1b_decode_step(self, k: torch.Tensor, v: torch.Tensor, q: torch.Tensor, inv_tau: float,
                        out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
        """Append one token per sequence to every layer and decode: k, v fp16 CUDA [L, B, 1, Hkv, d],
        q fp16 CUDA [L, B, Hq, d] -> out fp32 [L, B, Hq, d]."""
        kp, vp, qp = _dev_ptr(k, torch.float16, "k"), _dev_ptr(v, torch.float16, "v"), _dev_ptr(q, torch.float16, "q")
        L, B = self.cfg.n_layers, int(q.shape[1])
        if tuple(k.shape) != (L, B, 1, self.cfg.n_kv_heads, self.cfg.head_dim) or k.shape != v.shape or \
                tuple(q.shape) != (L, B, self.cfg.n_q_heads, self.cfg.head_dim):
            raise ValueError("step shapes: k, v [L, B, 1, Hkv, d]; q [L, B, Hq, d]")
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
        op = _dev_ptr(out, torch.float32, "out")
        self._check(self.lib.h1b_decode_step(self._h, kp, vp, qp, float(inv_tau), op, B, _stream_ptr(stream)))
        return out

    def h1b_decode_step_layers(self, layer_begin: int, k: torch.Tensor, v: torch.Tensor, q: torch.Tensor,
                               inv_tau: float, out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
        """The step for layers [layer_begin, layer_begin + n): k, v fp16 CUDA [n, B, 1, Hkv, d],
        q fp16 CUDA [n, B, Hq, d] -> out fp32 [n, B, Hq, d]."""
        kp, vp, qp = _dev_ptr(k, torch.float16, "k"), _dev_ptr(v, torch.float16, "v"), _dev_ptr(q, torch.float16, "q")
        n, B = int(q.shape[0]), int(q.shape[1])
        if tuple(k.shape) != (n, B, 1, self.cfg.n_kv_heads, self.cfg.head_dim) or k.shape != v.shape or \
                tuple(q.shape) != (n, B, self.cfg.n_q_heads, self.cfg.head_dim):
            raise ValueError("step shapes: k, v [n, B, 1, Hkv, d]; q [n, B, Hq, d]")
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
        op = _dev_ptr(out, torch.float32, "out")
        self._check(self.lib.h1b_decode_step_layers(self._h, layer_begin, n, kp, vp, qp, float(inv_tau), op, B,
                                                    _stream_ptr(stream)))
        return out

    def h1b_set_block_table(self, seq: int, pages, stream=None):
        """Paged cache: sequence `seq` owns these pool pages, in this order."""
        arr = np.ascontiguousarray(pages, dtype=np.int32)
        self._check(self.lib.h1b_set_block_table(self._h, seq, arr.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                                 int(arr.size), _stream_ptr(stream)))

    def h1b_set_rope_table(self, cos_sin, stream=None):
        """Rotary table: cos_sin fp32 [n_positions, d/2, 2] (numpy or CPU tensor), (cos, sin) per position and pair."""
        arr = np.ascontiguousarray(cos_sin.numpy() if isinstance(cos_sin, torch.Tensor) else cos_sin, dtype=np.float32)
        if arr.ndim != 3 or arr.shape[1:] != (self.cfg.head_dim // 2, 2):
            raise ValueError("cos_sin must be [n_positions, d/2, 2]")
        self._check(self.lib.h1b_set_rope_table(self._h, arr.ctypes.data, int(arr.shape[0]), _stream_ptr(stream)))

    def h1b_sync_lengths(self, stream=None):
        """After replaying a captured graph that appends: refresh the host's copy of the lengths."""
        self._check(self.lib.h1b_sync_lengths(self._h, _stream_ptr(stream)))

    def h1b_decode_attention_static(self, q: torch.Tensor, inv_tau: float, out: torch.Tensor,
                                    layer_begin: int = 0, stream=None) -> torch.Tensor:
        """h1b_decode_attention for callers that must not allocate: the temporaries live in the
        library's built-in 8 MiB device array, and `out` has to be supplied (nothing is created
        here either). q fp16 CUDA [n_layers, B, Hq, d], out fp32 CUDA of the same shape. The
        context's device must be current; calls that overlap on the GPU race on the shared array."""
        qp = _dev_ptr(q, torch.float16, "q")
        op = _dev_ptr(out, torch.float32, "out")
        if q.dim() != 4 or q.shape[2] != self.cfg.n_q_heads or q.shape[3] != self.cfg.head_dim or out.shape != q.shape:
            raise ValueError("q and out must be [n_layers, B, Hq, d]")
        self._check(self.lib.h1b_decode_attention_static(self._h, layer_begin, int(q.shape[0]), qp, float(inv_tau),
                                                         op, int(q.shape[1]), _stream_ptr(stream)))
        return out

    def h1b_decode_step_host(self, k: torch.Tensor, v: torch.Tensor, q: torch.Tensor, inv_tau: float,
                             out: torch.Tensor, stream=None) -> torch.Tensor:
        """Host tensors (pinned for asynchronous copies): k, v fp16 [L, B, 1, Hkv, d], q fp16 [L, B, Hq, d],
        out fp32 [L, B, Hq, d]. Copies, appends, decodes, copies back, synchronises."""
        for t, dt, name in ((k, torch.float16, "k"), (v, torch.float16, "v"), (q, torch.float16, "q"),
                            (out, torch.float32, "out")):
            if t.is_cuda or not t.is_contiguous() or t.dtype != dt:
                raise TypeError("%s must be a contiguous host tensor of dtype %s" % (name, dt))
        L, B = self.cfg.n_layers, int(q.shape[1])
        if tuple(k.shape) != (L, B, 1, self.cfg.n_kv_heads, self.cfg.head_dim) or k.shape != v.shape or \
                tuple(q.shape) != (L, B, self.cfg.n_q_heads, self.cfg.head_dim) or out.shape != q.shape:
            raise ValueError("host step shapes: k, v [L, B, 1, Hkv, d]; q, out [L, B, Hq, d]")
        self._check(self.lib.h1b_decode_step_host(self._h, k.data_ptr(), v.data_ptr(), q.data_ptr(), float(inv_tau),
                                                  out.data_ptr(), B, _stream_ptr(stream)))
        return out

    # -- introspection -----------------------------------------------------
    def h1b_get_projection(self, layer: int) -> np.ndarray:
        Rt = np.empty((self.cfg.head_dim, self.cfg.sketch_bits), dtype=np.float32)
        self._check(self.lib.h1b_get_projection(self._h, layer, Rt.ctypes.data))
        return Rt

    def h1b_get_lengths(self, layer: int) -> np.ndarray:
        ln = np.empty((self.cfg.max_batch,), dtype=np.int32)
        self._check(self.lib.h1b_get_lengths(self._h, layer, ln.ctypes.data))
        return ln

    def h1b_reset(self, seq: int = -1):
        self._check(self.lib.h1b_reset(self._h, seq))

    def h1b_truncate(self, seq: int, new_len: int):
        self._check(self.lib.h1b_truncate(self._h, seq, new_len))

    def h1b_truncate_async(self, seq: int, new_len: int, stream=None):
        """h1b_truncate ordered on the stream, without waiting for the device."""
        self._check(self.lib.h1b_truncate_async(self._h, seq, new_len, _stream_ptr(stream)))

    def h1b_export_cache(self, layer: int, seq: int, kv_head: int, t0: int, n: int):
        """-> (words uint32 [n, m/32], codes uint8 [n, d], scale uint16 [n, d/G], zero uint16 [n, d/G])."""
        c = self.cfg
        words = np.empty((n, c.sketch_bits // 32), dtype=np.uint32)
        if c.flags & H1B_FLAG_FP16_VALUES:              # no codes, scales or zero-points in this cache
            self._check(self.lib.h1b_export_cache(self._h, layer, seq, kv_head, t0, n, words.ctypes.data,
                                                  None, None, None))
            return words, None, None, None
        codes = np.empty((n, c.head_dim), dtype=np.uint8)
        scale = np.empty((n, c.head_dim // c.group_size), dtype=np.uint16)
        zero = np.empty_like(scale)
        self._check(self.lib.h1b_export_cache(self._h, layer, seq, kv_head, t0, n, words.ctypes.data,
                                              codes.ctypes.data, scale.ctypes.data, zero.ctypes.data))
        return words, codes, scale, zero

    def h1b_export_values(self, layer: int, seq: int, kv_head: int, t0: int, n: int) -> np.ndarray:
        """fp16-value caches only -> values uint16 [n, d] (fp16 bit patterns)."""
        values = np.empty((n, self.cfg.head_dim), dtype=np.uint16)
        self._check(self.lib.h1b_export_values(self._h, layer, seq, kv_head, t0, n, values.ctypes.data))
        return values

    def h1b_debug_scores(self, layer: int, seq: int, kv_head: int, q_row: torch.Tensor, n_tokens: int):
        """q_row: fp16 CUDA [d]. -> (qwords uint32 [m/32], score int32 [n_tokens])."""
        qp = _dev_ptr(q_row, torch.float16, "q_row")
        qwords = np.empty((self.cfg.sketch_bits // 32,), dtype=np.uint32)
        score = np.empty((max(n_tokens, 1),), dtype=np.int32)
        self._check(self.lib.h1b_debug_scores(self._h, layer, seq, kv_head, qp, qwords.ctypes.data, score.ctypes.data))
        return qwords, score[:n_tokens]

    def h1b_debug_partials(self, layer: int, seq: int, q_token: int, q_head: int, max_splits: int = 4096):
        """After an attention call: (hmin float32 [S], wsum float32 [S]) of the last launch's splits for one head."""
        n = ctypes.c_int32()
        hmin = np.empty((max_splits,), dtype=np.float32)
        wsum = np.empty((max_splits,), dtype=np.float32)
        self._check(self.lib.h1b_debug_partials(self._h, layer, seq, q_token, q_head, ctypes.byref(n), hmin.ctypes.data,
                                                wsum.ctypes.data, max_splits))
        return hmin[:n.value].copy(), wsum[:n.value].copy()

    def h1b_debug_prompt_scores(self, layer: int, seq: int, q_head: int, score_dev, n_tokens: int):
        """The next tile-route h1b_prefill_attention call exports one head's integer scores to score_dev (int32 CUDA [Tn, n_tokens])."""
        ptr = None if score_dev is None else _dev_ptr(score_dev, torch.int32, "score_dev")
        self._check(self.lib.h1b_debug_prompt_scores(self._h, layer, seq, q_head, ptr, n_tokens))

    def h1b_debug_prompt_route(self, tiles: bool):
        """False: prompt attention walks 16 query tokens at a time through the decode kernels, whatever the run's length."""
        self._check(self.lib.h1b_debug_prompt_route(self._h, int(bool(tiles))))

    def h1b_debug_prompt_stall(self, limit_ns: int):
        """The next tile-route h1b_prefill_attention call runs with its issuing warp idle and waits limited to limit_ns:
        its row threads time out, the next h1b_poll_status() reports it (the call's output is undefined)."""
        self._check(self.lib.h1b_debug_prompt_stall(self._h, int(limit_ns)))

    def h1b_debug_bounds_probe(self, stream=None):
        """Bounds-checked build only: a kernel's check fails on purpose; the next h1b_poll_status() reports it."""
        self._check(self.lib.h1b_debug_bounds_probe(self._h, _stream_ptr(stream)))

    def h1b_debug_wait_timeout(self, limit_ns: int, stream=None):
        """Failure-path probe: one warp's bounded wait runs out and is recorded in the status word."""
        self._check(self.lib.h1b_debug_wait_timeout(self._h, int(limit_ns), _stream_ptr(stream)))

    def h1b_set_splits(self, splits: int):
        self._check(self.lib.h1b_set_splits(self._h, splits))

    def h1b_poll_status(self):
        self._check(self.lib.h1b_poll_status(self._h))

    def h1b_set_profiling(self, enable: bool):
        self._check(self.lib.h1b_set_profiling(self._h, int(bool(enable))))

    def h1b_read_profile(self):
        """-> (summed split-K kernel time in ms, number of recorded launches)."""
        ms, n = ctypes.c_double(), ctypes.c_int64()
        self._check(self.lib.h1b_read_profile(self._h, ctypes.byref(ms), ctypes.byref(n)))
        return float(ms.value), int(n.value)

    def h1b_launch_count(self) -> int:
        return int(self.lib.h1b_launch_count(self._h))


def unpack_words(words: np.ndarray, m: int) -> np.ndarray:
    """uint32 [n, m/32] -> bits uint8 [n, m] (bit j = bit j%32 of word j/32). Marshalling only."""
    w = np.ascontiguousarray(words, dtype=np.uint32)
    bits = ((w[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1).astype(np.uint8)
    return bits.reshape(w.shape[0], m)
