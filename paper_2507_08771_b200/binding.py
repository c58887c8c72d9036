"""Python binding of the BlockFFN C-ABI library (argument marshalling only).

Each ``blockffn_*`` function below has the name and argument order of the C entry
point in ``include/blockffn.h``; tensors are torch CUDA tensors whose raw device
pointers are handed over, streams are torch streams. All computation happens in
the CUDA library: there is no fallback, and loading fails loudly if the shared
object has not been built (``python __graft_entry__.py``).
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libblockffn.so")
_lib = None

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_DEVICE = range(6)
DEV_BAD_UNION_ID, DEV_BAD_UNION_COUNT, DEV_WAIT_EXPIRED = 1, 2, 4
VARIANT_AUTO, VARIANT_SIMT, VARIANT_MMA = 0, 1, 2
CALL_ACCUMULATE, CALL_INDEPENDENT, CALL_INDEPENDENT_X = 1, 2, 4
CFG_NO_CHAINING = 0x10000
CFG_TWO_KERNELS = 0x20000000
CFG_TEST_EXPIRE_WAIT = 0x10000000
CFG_NO_SPLIT = 0x40000000
NO_RMSNORM = -1.0        # rms_eps value: the router without RMSNorm (Sec. 4.2.3)


def cfg_expected_union(u: int) -> int:
    """flags bits that tell the tensor-core kernels how large a union to size their stages for."""
    return (int(u) & 0x7ff) << 17

EXPORTS = [
    "blockffn_create", "blockffn_destroy", "blockffn_router", "blockffn_chunk_union",
    "blockffn_expert_ffn", "blockffn_layer_forward", "blockffn_layer_forward_scores",
    "blockffn_read_routing", "blockffn_last_status", "blockffn_tls", "blockffn_cls",
    "blockffn_launch_count", "blockffn_status_string", "blockffn_expert_ffn_noalloc",
    "blockffn_reuse_ratio",
]
NOALLOC_SCRATCH_BYTES = 1 << 20


class Config(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("E", ctypes.c_int32), ("d_e", ctypes.c_int32),
                ("L_max", ctypes.c_int32), ("rms_eps", ctypes.c_float),
                ("variant", ctypes.c_int32), ("flags", ctypes.c_int32)]


class Weights(ctypes.Structure):
    _fields_ = [("W_r", ctypes.c_void_p), ("gain", ctypes.c_void_p), ("bias", ctypes.c_void_p),
                ("U", ctypes.c_void_p), ("D", ctypes.c_void_p)]


class Stats(ctypes.Structure):
    _fields_ = [("n_tokens", ctypes.c_uint64), ("n_active", ctypes.c_uint64),
                ("n_chunks", ctypes.c_uint64), ("n_union", ctypes.c_uint64)]


class BlockFFNError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


def load():
    """Loads libblockffn.so (built in-tree). Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} not found: build it with `python __graft_entry__.py` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32 = ctypes.c_void_p, ctypes.c_int32
    lib.blockffn_create.argtypes = [ctypes.POINTER(Config), ctypes.POINTER(vp)]
    lib.blockffn_destroy.argtypes = [vp]
    lib.blockffn_router.argtypes = [vp, ctypes.POINTER(Weights), vp, i32, vp, vp, vp]
    lib.blockffn_chunk_union.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp]
    lib.blockffn_expert_ffn.argtypes = [vp, ctypes.POINTER(Weights), vp, vp, i32, vp, vp, vp, vp,
                                        i32, vp]
    lib.blockffn_layer_forward.argtypes = [vp, ctypes.POINTER(Weights), vp, i32, vp, vp, vp, i32, vp]
    lib.blockffn_layer_forward_scores.argtypes = [vp, ctypes.POINTER(Weights), vp, vp, i32, vp, vp,
                                                  vp, i32, vp]
    lib.blockffn_read_routing.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp]
    lib.blockffn_expert_ffn_noalloc.argtypes = [ctypes.POINTER(Config), ctypes.POINTER(Weights), vp,
                                                vp, i32, vp, vp, vp, vp, i32, vp]
    lib.blockffn_last_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32), i32, vp]
    lib.blockffn_tls.argtypes = [ctypes.POINTER(Stats), i32]
    lib.blockffn_tls.restype = ctypes.c_double
    lib.blockffn_cls.argtypes = [ctypes.POINTER(Stats), i32]
    lib.blockffn_cls.restype = ctypes.c_double
    lib.blockffn_reuse_ratio.argtypes = [vp, vp, i32, vp, vp]
    lib.blockffn_launch_count.argtypes = [vp]
    lib.blockffn_launch_count.restype = ctypes.c_uint64
    lib.blockffn_status_string.argtypes = [i32]
    lib.blockffn_status_string.restype = ctypes.c_char_p
    for name in EXPORTS:
        getattr(lib, name)
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load().blockffn_status_string(int(code)).decode()


def _ptr(t):
    """Raw device pointer of a tensor (or an int address, or None)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_cuda and t.is_contiguous(), "device tensors must be CUDA and contiguous"
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(code, where):
    if code != OK:
        raise BlockFFNError(code, where)


def make_weights(W_r=None, gain=None, bias=None, U=None, D=None) -> Weights:
    return Weights(_ptr(W_r), _ptr(gain), _ptr(bias), _ptr(U), _ptr(D))


# ---- entry points, same names as the C ABI ------------------------------------
def blockffn_create(d, E, d_e, L_max, rms_eps=1e-6, variant=VARIANT_AUTO, flags=0):
    cfg = Config(d, E, d_e, L_max, rms_eps, variant, flags)
    h = ctypes.c_void_p()
    _check(load().blockffn_create(ctypes.byref(cfg), ctypes.byref(h)), "blockffn_create")
    return h


def blockffn_destroy(h):
    _check(load().blockffn_destroy(h), "blockffn_destroy")


def blockffn_router(h, w: Weights, x, L, scores, tok_mask=None, stream=None):
    _check(load().blockffn_router(h, ctypes.byref(w), _ptr(x), L, _ptr(scores), _ptr(tok_mask),
                                  _stream(stream)), "blockffn_router")


def blockffn_chunk_union(h, scores, L, union_mask, union_ids, n_union, stats=None, stream=None):
    _check(load().blockffn_chunk_union(h, _ptr(scores), L, _ptr(union_mask), _ptr(union_ids),
                                       _ptr(n_union), _ptr(stats), _stream(stream)),
           "blockffn_chunk_union")


def blockffn_expert_ffn(h, w: Weights, x, scores, L, union_ids, n_union, out, x_next=None,
                        call_flags=0, stream=None):
    _check(load().blockffn_expert_ffn(h, ctypes.byref(w), _ptr(x), _ptr(scores), L,
                                      _ptr(union_ids), _ptr(n_union), _ptr(out), _ptr(x_next),
                                      call_flags, _stream(stream)), "blockffn_expert_ffn")


def blockffn_expert_ffn_noalloc(cfg: Config, w: Weights, x, scores, L, union_ids, n_union, out,
                                x_next=None, call_flags=0, stream=None):
    """Expert stage for callers that may not allocate device memory: no handle, the
    intermediate lives in a fixed array inside the library (see the header for its limits)."""
    _check(load().blockffn_expert_ffn_noalloc(ctypes.byref(cfg), ctypes.byref(w), _ptr(x),
                                              _ptr(scores), L, _ptr(union_ids), _ptr(n_union),
                                              _ptr(out), _ptr(x_next), call_flags,
                                              _stream(stream)), "blockffn_expert_ffn_noalloc")


def blockffn_layer_forward(h, w: Weights, x, L, out, x_next=None, stats=None, call_flags=0,
                           stream=None):
    _check(load().blockffn_layer_forward(h, ctypes.byref(w), _ptr(x), L, _ptr(out), _ptr(x_next),
                                         _ptr(stats), call_flags, _stream(stream)),
           "blockffn_layer_forward")


def blockffn_layer_forward_scores(h, w: Weights, x, scores, L, out, x_next=None, stats=None,
                                  call_flags=0, stream=None):
    _check(load().blockffn_layer_forward_scores(h, ctypes.byref(w), _ptr(x), _ptr(scores), L,
                                                _ptr(out), _ptr(x_next), _ptr(stats), call_flags,
                                                _stream(stream)), "blockffn_layer_forward_scores")


def blockffn_read_routing(h, L, scores=None, tok_mask=None, union_mask=None, union_ids=None,
                          n_union=None, stream=None):
    _check(load().blockffn_read_routing(h, L, _ptr(scores), _ptr(tok_mask), _ptr(union_mask),
                                        _ptr(union_ids), _ptr(n_union), _stream(stream)),
           "blockffn_read_routing")


def blockffn_reuse_ratio(h, scores, L, reuse, stream=None):
    _check(load().blockffn_reuse_ratio(h, _ptr(scores), L, _ptr(reuse), _stream(stream)),
           "blockffn_reuse_ratio")


def blockffn_last_status(h, clear=False, stream=None) -> int:
    bits = ctypes.c_uint32(0)
    code = load().blockffn_last_status(h, ctypes.byref(bits), int(clear), _stream(stream))
    if code not in (OK, ERR_DEVICE):
        raise BlockFFNError(code, "blockffn_last_status")
    return int(bits.value)


def blockffn_tls(stats_host: Stats, E: int) -> float:
    return float(load().blockffn_tls(ctypes.byref(stats_host), E))


def blockffn_cls(stats_host: Stats, E: int) -> float:
    return float(load().blockffn_cls(ctypes.byref(stats_host), E))


def blockffn_launch_count(h) -> int:
    return int(load().blockffn_launch_count(h))


# ---- small conveniences for tests and the benchmark (no arithmetic) ------------
def to_device_bf16(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bf16 bit patterns (numpy) -> torch.bfloat16 CUDA tensor of the same shape."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)


def stats_to_host(stats_dev: torch.Tensor) -> Stats:
    v = stats_dev.cpu().numpy().view(np.uint64)
    return Stats(int(v[0]), int(v[1]), int(v[2]), int(v[3]))


@dataclass
class DeviceWeights:
    struct: Weights
    tensors: dict      # keeps the device tensors alive


@dataclass
class LayerOutput:
    out: torch.Tensor          # f32 [L][d]
    scores: torch.Tensor       # f32 [L][E]
    tok_mask: torch.Tensor | None
    union_mask: torch.Tensor   # i32 view of u32 [W]
    union_ids: torch.Tensor    # i32 [E]
    n_union: torch.Tensor      # i32 [1]


class Layer:
    """Owns one library handle and output buffers; forwards to the C entry points."""

    def __init__(self, d, E, d_e, L_max=32, rms_eps=1e-6, variant=VARIANT_AUTO, device="cuda",
                 flags=0):
        self.d, self.E, self.d_e, self.L_max = d, E, d_e, L_max
        self.words = (E + 31) // 32
        self.device = torch.device(device)
        self.h = blockffn_create(d, E, d_e, L_max, rms_eps, variant, flags)
        self.stats = torch.zeros(4, dtype=torch.int64, device=self.device)

    def close(self):
        if self.h is not None:
            torch.cuda.synchronize()
            blockffn_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def upload_weights(self, w: dict) -> DeviceWeights:
        t = {}
        for k in ("W_r", "U", "D"):
            if w.get(k) is not None:
                t[k] = to_device_bf16(w[k], self.device)
        for k in ("gain", "bias"):
            if w.get(k) is not None:
                t[k] = torch.from_numpy(np.ascontiguousarray(w[k], dtype=np.float32)).to(self.device)
        return DeviceWeights(make_weights(t.get("W_r"), t.get("gain"), t.get("bias"), t.get("U"),
                                          t.get("D")), t)

    def _routing(self, L, with_scores):
        """What the last layer call derived, copied out of the handle's workspace."""
        dev = self.device
        scores = torch.empty(L, self.E, dtype=torch.float32, device=dev) if with_scores else None
        tok = torch.empty(L, self.words, dtype=torch.int32, device=dev) if with_scores else None
        um = torch.empty(self.words, dtype=torch.int32, device=dev)
        ids = torch.empty(self.E, dtype=torch.int32, device=dev)
        nu = torch.empty(1, dtype=torch.int32, device=dev)
        blockffn_read_routing(self.h, L, scores, tok, um, ids, nu)
        return scores, tok, um, ids, nu

    def forward(self, dw: DeviceWeights, x: torch.Tensor, out=None, x_next=None, call_flags=0,
                stream=None) -> LayerOutput:
        L = x.shape[0]
        if out is None:
            out = torch.empty(L, self.d, dtype=torch.float32, device=self.device)
        blockffn_layer_forward(self.h, dw.struct, x, L, out, x_next, self.stats, call_flags, stream)
        scores, tok, um, ids, nu = self._routing(L, True)
        return LayerOutput(out, scores, tok, um, ids, nu)

    def forward_scores(self, dw: DeviceWeights, x: torch.Tensor, scores: torch.Tensor, out=None,
                       x_next=None, call_flags=0, stream=None) -> LayerOutput:
        L = x.shape[0]
        if out is None:
            out = torch.empty(L, self.d, dtype=torch.float32, device=self.device)
        blockffn_layer_forward_scores(self.h, dw.struct, x, scores, L, out, x_next, self.stats,
                                      call_flags, stream)
        _, _, um, ids, nu = self._routing(L, False)
        return LayerOutput(out, scores, None, um, ids, nu)

    def last_status(self, clear=False) -> int:
        return blockffn_last_status(self.h, clear)

    def launch_count(self) -> int:
        return blockffn_launch_count(self.h)

    def stats_host(self) -> Stats:
        return stats_to_host(self.stats)
