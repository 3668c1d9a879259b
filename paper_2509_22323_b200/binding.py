"""ctypes binding of librapid3.so: argument marshalling only.

Every step of the path runs in the CUDA kernels behind the C ABI (include/rapid3.h); torch is
used for device memory and streams.  There is no CPU fallback: if the shared library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "librapid3.so")

OK = 0
ACT_SKIP, ACT_REUSE, ACT_ATTEND = 0, 1, 2

EXPORTS = [
    "rapid3_create", "rapid3_destroy", "rapid3_strerror", "rapid3_num_blocks", "rapid3_mask_words",
    "rapid3_block_scores", "rapid3_select_mask", "rapid3_sparse_joint_attn", "rapid3_gated_step",
    "rapid3_gated_step_host", "rapid3_workspace", "rapid3_launch_count", "rapid3_last_status",
    "rapid3_profile", "rapid3_profile_read", "rapid3_block_scores_static", "rapid3_static_scratch_bytes", "rapid3_cache_step", "rapid3_gated_step_device", "rapid3_gated_step_heads", "rapid3_equivalent_steps", "rapid3_select_mask_mass", "rapid3_gated_step_fused", "rapid3_gated_step_mass",
    "rapid3_debug_inject_timeout",
]


class Rapid3Error(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} ({code})")
        self.code = code


class Shape(ctypes.Structure):
    _fields_ = [("B_max", ctypes.c_int32), ("H", ctypes.c_int32), ("D", ctypes.c_int32),
                ("n_text", ctypes.c_int32), ("n_image", ctypes.c_int32), ("block", ctypes.c_int32),
                ("stride_b", ctypes.c_int64), ("stride_h", ctypes.c_int64), ("stride_n", ctypes.c_int64)]


_lib = None


def load() -> ctypes.CDLL:
    """Loads librapid3.so (built in-tree by paper_2509_22323_b200.build); raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} not found: build the CUDA library first (python -m paper_2509_22323_b200.build); "
            "there is no CPU fallback")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    i32p, f32p, i64p = ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int64)
    lib.rapid3_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(Shape)]
    lib.rapid3_destroy.argtypes = [vp]
    lib.rapid3_strerror.argtypes = [ci]
    lib.rapid3_strerror.restype = ctypes.c_char_p
    lib.rapid3_num_blocks.argtypes = [ctypes.POINTER(Shape)]
    lib.rapid3_mask_words.argtypes = [ctypes.POINTER(Shape)]
    lib.rapid3_block_scores.argtypes = [vp, vp, vp, i32p, ci, vp, vp]
    lib.rapid3_select_mask.argtypes = [vp, vp, f32p, ci, vp, vp, vp, vp]
    lib.rapid3_select_mask_mass.argtypes = [vp, vp, f32p, cf, ci, vp, vp, vp, vp, vp]
    lib.rapid3_sparse_joint_attn.argtypes = [vp, vp, vp, vp, vp, i32p, ci, vp, vp, cf, vp]
    lib.rapid3_gated_step.argtypes = [vp, vp, vp, vp, vp, i32p, f32p, ci, cf, vp]
    lib.rapid3_gated_step_fused.argtypes = [vp, vp, vp, vp, vp, vp, vp, cf, vp, vp, vp, i32p, f32p, ci, cf, vp]
    lib.rapid3_gated_step_mass.argtypes = [vp, vp, vp, vp, vp, i32p, f32p, cf, ci, cf, vp]
    lib.rapid3_gated_step_heads.argtypes = [vp, vp, vp, vp, vp, i32p, f32p, ci, cf, vp]
    lib.rapid3_gated_step_device.argtypes = [vp, vp, vp, vp, vp, vp, vp, ci, cf, vp]
    lib.rapid3_gated_step_host.argtypes = [vp, vp, vp, vp, vp, i32p, f32p, ci, cf, vp, i64p, i64p]
    lib.rapid3_debug_inject_timeout.argtypes = [vp, vp, vp, vp, vp, ci, cf, vp]
    lib.rapid3_workspace.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp)]
    lib.rapid3_launch_count.argtypes = [vp]
    lib.rapid3_launch_count.restype = ctypes.c_int64
    lib.rapid3_last_status.argtypes = [vp, ctypes.POINTER(ci)]
    lib.rapid3_profile.argtypes = [vp, ci]
    lib.rapid3_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_double), i64p]
    lib.rapid3_block_scores_static.argtypes = [ctypes.POINTER(Shape), vp, vp, i32p, ci, vp, vp]
    lib.rapid3_static_scratch_bytes.argtypes = []
    lib.rapid3_equivalent_steps.argtypes = [i32p, f32p, f32p, ci, ctypes.POINTER(ctypes.c_double), i64p]
    lib.rapid3_cache_step.argtypes = [vp, vp, vp, i32p, ci, ctypes.c_int64, vp]
    lib.rapid3_static_scratch_bytes.restype = ctypes.c_int64
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().rapid3_strerror(int(code)).decode()


def _check(code: int, what: str):
    if code != OK:
        raise Rapid3Error(code, what)


def _i32(xs: Optional[Sequence[int]]):
    if xs is None:
        return None
    return (ctypes.c_int32 * len(xs))(*[int(x) for x in xs])


def _f32(xs: Sequence[float]):
    return (ctypes.c_float * len(xs))(*[float(x) for x in xs])


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


class Context:
    """Owns a rapid3_ctx for tensors of shape [B<=B_max, H, N, D] with the given element strides."""

    def __init__(self, B_max: int, H: int, D: int, n_text: int, n_image: int,
                 strides: Optional[Sequence[int]] = None):
        self.lib = load()
        N = n_text + n_image
        if strides is None:
            strides = (H * N * D, N * D, D)
        self.shape = Shape(B_max, H, D, n_text, n_image, 64, int(strides[0]), int(strides[1]), int(strides[2]))
        self.B_max, self.H, self.D, self.n_text, self.n_image, self.N = B_max, H, D, n_text, n_image, N
        self.handle = ctypes.c_void_p()
        _check(self.lib.rapid3_create(ctypes.byref(self.handle), ctypes.byref(self.shape)), "rapid3_create")
        self.nb = self.lib.rapid3_num_blocks(ctypes.byref(self.shape))
        self.words = self.lib.rapid3_mask_words(ctypes.byref(self.shape))

    def close(self):
        if getattr(self, "handle", None) is not None and self.handle.value:
            self.lib.rapid3_destroy(self.handle)
            self.handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the four calls of the path (same names as the C ABI) ----
    def rapid3_block_scores(self, q: torch.Tensor, k: torch.Tensor, img_idx: Optional[Sequence[int]] = None,
                            n_img: Optional[int] = None, scores: Optional[torch.Tensor] = None) -> torch.Tensor:
        n = len(img_idx) if img_idx is not None else (n_img if n_img is not None else q.shape[0])
        if scores is None:
            scores = torch.empty((n, self.H, self.nb, self.nb), dtype=torch.float32, device=q.device)
        _check(self.lib.rapid3_block_scores(self.handle, _ptr(q), _ptr(k), _i32(img_idx), n, _ptr(scores), _stream()),
               "rapid3_block_scores")
        return scores

    def rapid3_select_mask(self, scores: torch.Tensor, keep_ratio: Sequence[float], out=None):
        n = len(keep_ratio)
        dev = scores.device
        if out is None:
            bitmask = torch.empty((n, self.H, self.nb, self.words), dtype=torch.int64, device=dev)
            kept_idx = torch.empty((n, self.H, self.nb, self.nb), dtype=torch.int32, device=dev)
            kept_cnt = torch.empty((n, self.H, self.nb), dtype=torch.int32, device=dev)
        else:
            bitmask, kept_idx, kept_cnt = out
        _check(self.lib.rapid3_select_mask(self.handle, _ptr(scores), _f32(keep_ratio), n, _ptr(bitmask),
                                           _ptr(kept_idx), _ptr(kept_cnt), _stream()), "rapid3_select_mask")
        return bitmask, kept_idx, kept_cnt

    def rapid3_select_mask_mass(self, scores: torch.Tensor, mass_share: Sequence[float], mass_scale: float):
        """Cumulative-mass selection: returns (row_keep, bitmask, kept_idx, kept_cnt)."""
        n = scores.shape[0]
        assert len(mass_share) == n and scores.dtype == torch.float32 and scores.is_contiguous()
        dev = scores.device
        row_keep = torch.empty((n, self.H, self.nb), dtype=torch.int32, device=dev)
        bitmask = torch.empty((n, self.H, self.nb, self.words), dtype=torch.int64, device=dev)
        kept_idx = torch.empty((n, self.H, self.nb, self.nb), dtype=torch.int32, device=dev)
        kept_cnt = torch.empty((n, self.H, self.nb), dtype=torch.int32, device=dev)
        _check(self.lib.rapid3_select_mask_mass(self.handle, _ptr(scores), _f32(mass_share), float(mass_scale), n,
                                                _ptr(row_keep), _ptr(bitmask), _ptr(kept_idx), _ptr(kept_cnt),
                                                _stream()), "rapid3_select_mask_mass")
        return row_keep, bitmask, kept_idx, kept_cnt

    def rapid3_sparse_joint_attn(self, q, k, v, out, img_idx: Optional[Sequence[int]] = None,
                                 n_img: Optional[int] = None, kept_idx=None, kept_cnt=None,
                                 softmax_scale: Optional[float] = None):
        n = len(img_idx) if img_idx is not None else (n_img if n_img is not None else q.shape[0])
        scale = softmax_scale if softmax_scale is not None else self.D ** -0.5
        _check(self.lib.rapid3_sparse_joint_attn(self.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _i32(img_idx), n,
                                                 _ptr(kept_idx), _ptr(kept_cnt), scale, _stream()),
               "rapid3_sparse_joint_attn")
        return out

    def rapid3_gated_step(self, q, k, v, out, actions: Sequence[int], keep_ratio: Sequence[float],
                          softmax_scale: Optional[float] = None):
        scale = softmax_scale if softmax_scale is not None else self.D ** -0.5
        _check(self.lib.rapid3_gated_step(self.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _i32(actions),
                                          _f32(keep_ratio), len(actions), scale, _stream()), "rapid3_gated_step")
        return out

    def rapid3_gated_step_fused(self, q_raw, k_raw, v, q_gain, k_gain, rot, eps: float, q, k, out,
                                actions: Sequence[int], keep_ratio: Sequence[float],
                                softmax_scale: Optional[float] = None):
        """q_raw, k_raw -> (RMS norm, gain, rotary) -> q, k (may alias the raw tensors), then the gated step."""
        scale = softmax_scale if softmax_scale is not None else self.D ** -0.5
        assert q_gain.dtype == torch.float32 and k_gain.dtype == torch.float32
        assert rot is None or (rot.dtype == torch.float32 and rot.is_contiguous())
        _check(self.lib.rapid3_gated_step_fused(self.handle, _ptr(q_raw), _ptr(k_raw), _ptr(v), _ptr(q_gain),
                                                _ptr(k_gain), _ptr(rot), float(eps), _ptr(q), _ptr(k), _ptr(out),
                                                _i32(actions), _f32(keep_ratio), len(actions), scale, _stream()),
               "rapid3_gated_step_fused")
        return out

    def rapid3_gated_step_mass(self, q, k, v, out, actions: Sequence[int], mass_share: Sequence[float],
                               mass_scale: float, softmax_scale: Optional[float] = None):
        """The gated step with the cumulative-mass selection (share per image) instead of top-k."""
        scale = softmax_scale if softmax_scale is not None else self.D ** -0.5
        _check(self.lib.rapid3_gated_step_mass(self.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _i32(actions),
                                               _f32(mass_share), float(mass_scale), len(actions), scale, _stream()),
               "rapid3_gated_step_mass")
        return out

    def rapid3_gated_step_heads(self, q, k, v, out, actions: Sequence[int], keep_ratio: Sequence[Sequence[float]],
                                softmax_scale: Optional[float] = None):
        """keep_ratio: [B][H], one ratio per image and head."""
        scale = softmax_scale if softmax_scale is not None else self.D ** -0.5
        flat = [float(r) for row in keep_ratio for r in row]
        assert len(flat) == len(actions) * self.H
        _check(self.lib.rapid3_gated_step_heads(self.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _i32(actions),
                                                _f32(flat), len(actions), scale, _stream()),
               "rapid3_gated_step_heads")
        return out

    def rapid3_gated_step_device(self, q, k, v, out, actions_dev: torch.Tensor, keep_ratio_dev: torch.Tensor,
                                 softmax_scale: Optional[float] = None):
        """actions_dev: int32 [B], keep_ratio_dev: float32 [B], both on the GPU; no host read-back."""
        assert actions_dev.dtype == torch.int32 and keep_ratio_dev.dtype == torch.float32
        scale = softmax_scale if softmax_scale is not None else self.D ** -0.5
        _check(self.lib.rapid3_gated_step_device(self.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(actions_dev),
                                                 _ptr(keep_ratio_dev), int(actions_dev.numel()), scale, _stream()),
               "rapid3_gated_step_device")
        return out

    def rapid3_gated_step_host(self, q, k, v, out, actions: Sequence[int], keep_ratio: Sequence[float],
                               softmax_scale: Optional[float] = None):
        """q, k, v, out: contiguous HOST bf16 tensors [B, H, N, D] (pinned for asynchronous copies)."""
        scale = softmax_scale if softmax_scale is not None else self.D ** -0.5
        up, down = ctypes.c_int64(0), ctypes.c_int64(0)
        _check(self.lib.rapid3_gated_step_host(self.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _i32(actions),
                                               _f32(keep_ratio), len(actions), scale, _stream(),
                                               ctypes.byref(up), ctypes.byref(down)), "rapid3_gated_step_host")
        return up.value, down.value

    def rapid3_debug_inject_timeout(self, q, k, v, out, stop_group: int, softmax_scale: Optional[float] = None):
        """Test aid: dense attention over image 0 with the failure-injection build of the kernel."""
        scale = softmax_scale if softmax_scale is not None else self.D ** -0.5
        _check(self.lib.rapid3_debug_inject_timeout(self.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(out), int(stop_group),
                                                    scale, _stream()), "rapid3_debug_inject_timeout")

    # ---- helpers ----
    def workspace(self, n_sparse: int, device="cuda"):
        """Views (no copy) of the scores / bitmask / kept lists the last gated step wrote."""
        ptrs = [ctypes.c_void_p() for _ in range(4)]
        _check(self.lib.rapid3_workspace(self.handle, *[ctypes.byref(p) for p in ptrs]), "rapid3_workspace")
        shapes = [((n_sparse, self.H, self.nb, self.nb), torch.float32),
                  ((n_sparse, self.H, self.nb, self.words), torch.int64),
                  ((n_sparse, self.H, self.nb, self.nb), torch.int32),
                  ((n_sparse, self.H, self.nb), torch.int32)]
        return [_view(p.value, s, d, device) for p, (s, d) in zip(ptrs, shapes)]

    def launch_count(self) -> int:
        return int(self.lib.rapid3_launch_count(self.handle))

    def profile(self, enable):
        """False / 0: off; True / 1: an event pair around every launch; 2: around the attention kernel only."""
        _check(self.lib.rapid3_profile(self.handle, int(enable)), "rapid3_profile")

    def profile_read(self):
        """Summed device milliseconds and launch counts per kernel kind since the last read."""
        ms = (ctypes.c_double * 4)()
        n = (ctypes.c_int64 * 4)()
        _check(self.lib.rapid3_profile_read(self.handle, ms, n), "rapid3_profile_read")
        kinds = ("block_pool", "block_scores", "select_mask", "attention")
        return {k: (ms[i], n[i]) for i, k in enumerate(kinds)}

    def last_status(self) -> int:
        v = ctypes.c_int(0)
        _check(self.lib.rapid3_last_status(self.handle, ctypes.byref(v)), "rapid3_last_status")
        return v.value


def rapid3_block_scores_static(shape: Shape, q: torch.Tensor, k: torch.Tensor, scores: torch.Tensor,
                               img_idx: Optional[Sequence[int]] = None, n_img: Optional[int] = None) -> torch.Tensor:
    """Context-free scoring pass for hosts that may not allocate device memory: the block means go
    to the fixed array inside the library instead of a workspace.  `scores` ([n, H, nb, nb] fp32,
    device) is supplied by the caller; nothing is allocated here either."""
    n = len(img_idx) if img_idx is not None else (n_img if n_img is not None else q.shape[0])
    _check(load().rapid3_block_scores_static(ctypes.byref(shape), _ptr(q), _ptr(k), _i32(img_idx), n, _ptr(scores),
                                             _stream()), "rapid3_block_scores_static")
    return scores


def rapid3_equivalent_steps(actions: Sequence[int], c_cache: Sequence[float], c_sparse: Sequence[float]):
    """Equivalent steps K of one trajectory: (exact sum, nearest integer)."""
    n = len(actions)
    assert len(c_cache) == n and len(c_sparse) == n
    k, kr = ctypes.c_double(0.0), ctypes.c_int64(0)
    _check(load().rapid3_equivalent_steps(_i32(actions), _f32(c_cache), _f32(c_sparse), n, ctypes.byref(k),
                                          ctypes.byref(kr)), "rapid3_equivalent_steps")
    return k.value, kr.value


def rapid3_cache_step(x: torch.Tensor, o: torch.Tensor, delta: torch.Tensor, actions: Sequence[int]):
    """Cache-Reuse data path over a batch [B, ...] of contiguous bf16 tensors: refreshes `delta` for
    attending images, writes `o` for reusing ones, leaves skipped ones alone."""
    B = len(actions)
    elems = x[0].numel()
    _check(load().rapid3_cache_step(_ptr(x), _ptr(o), _ptr(delta), _i32(actions), B, elems, _stream()),
           "rapid3_cache_step")


def static_scratch_bytes() -> int:
    return int(load().rapid3_static_scratch_bytes())


class _Raw:
    """Minimal __cuda_array_interface__ carrier so torch can view library-owned device memory."""

    def __init__(self, ptr, shape, typestr):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (ptr, False), "version": 2}


def _view(ptr: int, shape, dtype, device):
    typestr = {torch.float32: "<f4", torch.int64: "<i8", torch.int32: "<i4"}[dtype]
    return torch.as_tensor(_Raw(ptr, shape, typestr), device=device)


def bitmask_to_dense(bitmask: torch.Tensor, nb: int) -> torch.Tensor:
    """[..., nb, words] int64 bitmask -> [..., nb, nb] uint8 (marshalling for tests and reports)."""
    bm = bitmask.cpu()
    j = torch.arange(nb)
    words = bm[..., (j // 64)]
    return ((words >> (j % 64)) & 1).to(torch.uint8)
