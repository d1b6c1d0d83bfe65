"""ctypes binding of libsparrow_attn: argument marshalling only.

Every step of the attention path runs in the library's CUDA kernels; torch is used here for device
memory and streams.  The functions carry the C ABI's names and argument order.  There is no CPU
fallback: if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsparrow_attn.so")

STATUS_NAMES = {0: "SPARROW_OK", 1: "SPARROW_ERR_NULL", 2: "SPARROW_ERR_SHAPE", 3: "SPARROW_ERR_TREE",
                4: "SPARROW_ERR_ANCHOR", 5: "SPARROW_ERR_WORKSPACE", 6: "SPARROW_ERR_CUDA",
                7: "SPARROW_ERR_TIMEOUT", 8: "SPARROW_ERR_ARCH"}

EXPORTS = ["sparrow_create", "sparrow_destroy", "sparrow_workspace_bytes", "sparrow_set_workspace",
           "sparrow_verify_attn", "sparrow_verify_attn_batch", "sparrow_anchor_attn",
           "sparrow_verify_step_host", "sparrow_verify_attn_static",
           "sparrow_build_ancestor_masks", "sparrow_build_anchor_idx",
           "sparrow_debug_ancestor_masks_device", "sparrow_debug_wait_counter", "sparrow_plan_splits",
           "sparrow_last_device_status", "sparrow_debug_status_word", "sparrow_launch_count",
           "sparrow_set_plan_policy", "sparrow_set_call_overlap", "sparrow_debug_early_trigger_copy",
           "sparrow_verify_attn_window", "sparrow_window_first_visible", "sparrow_window_first_visible_device",
           "sparrow_plan_target_items", "sparrow_anchor_attn_tree", "sparrow_kv_append", "sparrow_compact_anchors",
           "sparrow_hsr_fuse", "sparrow_accept_greedy", "sparrow_accept_sample", "sparrow_kv_keep_accepted", "sparrow_plan_piece_range",
           "sparrow_status_string"]


PLAN_LATENCY, PLAN_BALANCED, PLAN_THROUGHPUT = 0, 1, 2


class SparrowError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {STATUS_NAMES.get(status, status)}")


class Layout(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("kv_capacity", ctypes.c_int32),
                ("softmax_scale", ctypes.c_float), ("kv_stride_batch", ctypes.c_int64),
                ("kv_stride_head", ctypes.c_int64)]


_lib = None


def lib():
    """Loads the shared library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build it with "
                               "`python -m paper_2602_15318_b200.build` (there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        L.sparrow_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(Layout), ctypes.c_int]
        L.sparrow_destroy.argtypes = [vp]
        L.sparrow_workspace_bytes.argtypes = [vp, i32]
        L.sparrow_workspace_bytes.restype = ctypes.c_size_t
        L.sparrow_set_workspace.argtypes = [vp, vp, ctypes.c_size_t]
        L.sparrow_verify_attn.argtypes = [vp, vp, vp, vp, vp, vp, i32, vp, vp, vp]
        L.sparrow_verify_attn_batch.argtypes = [vp, vp, i32, vp]
        L.sparrow_verify_attn_window.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp]
        L.sparrow_window_first_visible.argtypes = [vp, i32, i32, i32, i32, vp, vp]
        L.sparrow_window_first_visible_device.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp]
        L.sparrow_verify_attn_static.argtypes = [ctypes.POINTER(Layout), vp, vp, vp, vp, vp, i32, vp, vp, vp]
        L.sparrow_anchor_attn.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp]
        L.sparrow_plan_piece_range.argtypes = [i32, i32, i32, vp, vp]
        L.sparrow_accept_greedy.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, vp]
        L.sparrow_hsr_fuse.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, vp, vp]
        L.sparrow_accept_sample.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp]
        L.sparrow_kv_keep_accepted.argtypes = [vp, vp, vp, vp, vp, vp, i32, vp]
        L.sparrow_kv_append.argtypes = [vp, vp, vp, vp, vp, vp, i32, vp]
        L.sparrow_compact_anchors.argtypes = [vp, vp, vp, vp, i32, vp, vp, i32, i32, vp]
        L.sparrow_anchor_attn_tree.argtypes = [vp, vp, vp, vp, vp, i32, i32, vp, i32, i32, vp, vp, vp]
        L.sparrow_verify_step_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp]
        L.sparrow_build_ancestor_masks.argtypes = [vp, i32, vp]
        L.sparrow_build_anchor_idx.argtypes = [i32, vp, i32, i32, i32, vp, vp]
        L.sparrow_debug_ancestor_masks_device.argtypes = [vp, vp, i32, vp, vp]
        L.sparrow_debug_wait_counter.argtypes = [vp, ctypes.c_uint32, vp]
        L.sparrow_plan_splits.argtypes = [i32, i32, i32, i32, vp, i32, vp, vp]
        L.sparrow_last_device_status.argtypes = [vp, vp]
        L.sparrow_set_plan_policy.argtypes = [vp, i32]
        L.sparrow_set_call_overlap.argtypes = [vp, i32]
        L.sparrow_debug_early_trigger_copy.argtypes = [vp, vp, vp, ctypes.c_size_t, ctypes.c_uint32, vp]
        L.sparrow_plan_target_items.argtypes = [vp]
        L.sparrow_plan_target_items.restype = i32
        L.sparrow_debug_status_word.argtypes = [vp]
        L.sparrow_debug_status_word.restype = ctypes.c_uint32
        L.sparrow_launch_count.argtypes = [vp]
        L.sparrow_launch_count.restype = i64
        L.sparrow_status_string.argtypes = [ctypes.c_int]
        L.sparrow_status_string.restype = ctypes.c_char_p
        for name in EXPORTS:
            if name not in ("sparrow_workspace_bytes", "sparrow_launch_count", "sparrow_status_string",
                            "sparrow_debug_status_word", "sparrow_plan_target_items"):
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def _chk(status: int, what: str):
    if status != 0:
        raise SparrowError(status, what)


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    return t.data_ptr()


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream or None
    return stream or None


def _i32_array(values: Sequence[int]):
    return (ctypes.c_int32 * len(values))(*[int(x) for x in values])


class Context:
    """Owns a sparrow_ctx and (by default) a torch-allocated workspace registered with it."""

    def __init__(self, batch: int, kv_capacity: int, kv_stride_batch: int, kv_stride_head: int,
                 softmax_scale: float, n_q_heads: int = 28, n_kv_heads: int = 4, head_dim: int = 128,
                 device: int = 0, max_T: int = 64, allocate_workspace: bool = True):
        self.layout = Layout(batch, n_q_heads, n_kv_heads, head_dim, kv_capacity, softmax_scale,
                             kv_stride_batch, kv_stride_head)
        self.device = device
        self.handle = ctypes.c_void_p()
        _chk(lib().sparrow_create(ctypes.byref(self.handle), ctypes.byref(self.layout), device),
             "sparrow_create")
        self.workspace = None
        if allocate_workspace:
            n = self.workspace_bytes(max_T)
            self.workspace = torch.empty(n, dtype=torch.uint8, device=f"cuda:{device}")
            self.set_workspace(self.workspace.data_ptr(), n)

    @classmethod
    def for_cache(cls, k_cache: torch.Tensor, softmax_scale: float, n_q_heads: int = 28, **kw):
        """Context matching a [B, Hkv, capacity, 128] bf16 cache tensor's strides."""
        assert k_cache.dim() == 4 and k_cache.stride(3) == 1 and k_cache.stride(2) == k_cache.shape[3]
        return cls(k_cache.shape[0], k_cache.shape[2], k_cache.stride(0), k_cache.stride(1),
                   softmax_scale, n_q_heads=n_q_heads, n_kv_heads=k_cache.shape[1],
                   head_dim=k_cache.shape[3], device=k_cache.device.index or 0, **kw)

    def workspace_bytes(self, max_T: int) -> int:
        return int(lib().sparrow_workspace_bytes(self.handle, max_T))

    def set_workspace(self, ptr: int, nbytes: int):
        _chk(lib().sparrow_set_workspace(self.handle, ptr, nbytes), "sparrow_set_workspace")

    def launch_count(self) -> int:
        return int(lib().sparrow_launch_count(self.handle))

    def last_device_status(self, stream=None) -> int:
        return int(lib().sparrow_last_device_status(self.handle, _stream_handle(stream)))

    def set_plan_policy(self, policy: int):
        _chk(lib().sparrow_set_plan_policy(self.handle, int(policy)), "sparrow_set_plan_policy")

    def set_call_overlap(self, enable: bool):
        """Single sparrow_verify_attn calls may start early behind this context's previous call."""
        _chk(lib().sparrow_set_call_overlap(self.handle, 1 if enable else 0), "sparrow_set_call_overlap")

    def plan_target_items(self) -> int:
        return int(lib().sparrow_plan_target_items(self.handle))

    def status_word(self) -> int:
        """Raw status word read by the last last_device_status() call (wait-site bits above bit 8)."""
        return int(lib().sparrow_debug_status_word(self.handle))

    def close(self):
        if self.handle:
            lib().sparrow_destroy(self.handle)
            self.handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def sparrow_verify_attn(ctx: Context, q, k_cache, v_cache, kv_len: Sequence[int], parents, T: int,
                        out, lse, stream=None):
    """q/out: CUDA bf16 [B,T,Hq,128]; caches: CUDA bf16; kv_len: host ints; parents: CUDA int32
    [B,T]; lse: CUDA fp32 [B,Hq,T]."""
    kl = _i32_array(kv_len)
    _chk(lib().sparrow_verify_attn(ctx.handle, _ptr(q), _ptr(k_cache), _ptr(v_cache), kl, _ptr(parents),
                                   T, _ptr(out), _ptr(lse), _stream_handle(stream)), "sparrow_verify_attn")


def sparrow_verify_attn_window(ctx: Context, q, k_cache, v_cache, kv_len: Sequence[int], parents, T_tree: int,
                               T_new: int, first_visible, first_visible_min: Optional[Sequence[int]], out, lse,
                               stream=None):
    """Verification kernel on a compacted anchored cache: queries = the last T_new of T_tree draft
    nodes; first_visible: CUDA int32 [B,T_new] or None; first_visible_min: host ints or None."""
    kl = _i32_array(kv_len)
    fm = _i32_array(first_visible_min) if first_visible_min is not None else None
    _chk(lib().sparrow_verify_attn_window(ctx.handle, _ptr(q), _ptr(k_cache), _ptr(v_cache), kl, _ptr(parents),
                                          T_tree, T_new, _ptr(first_visible), fm, _ptr(out), _ptr(lse),
                                          _stream_handle(stream)), "sparrow_verify_attn_window")


def sparrow_window_first_visible(anchor_idx: Sequence[int], window: int, T_tree: int, T_new: int):
    """Host helper: (first_visible list of T_new ints, their minimum)."""
    idx = _i32_array(anchor_idx)
    first = (ctypes.c_int32 * T_new)()
    lowest = ctypes.c_int32(0)
    _chk(lib().sparrow_window_first_visible(idx, len(anchor_idx), window, T_tree, T_new, first, ctypes.byref(lowest)),
         "sparrow_window_first_visible")
    return [int(x) for x in first], int(lowest.value)


def sparrow_window_first_visible_device(ctx: Context, anchor_idx, n_anchor: int, window: int, T_tree: int, T_new: int,
                                        first_visible, stream=None):
    _chk(lib().sparrow_window_first_visible_device(ctx.handle, _ptr(anchor_idx), n_anchor, window, T_tree, T_new,
                                                   _ptr(first_visible), _stream_handle(stream)),
         "sparrow_window_first_visible_device")


def sparrow_verify_attn_static(layout: Layout, q, k_cache, v_cache, kv_len: Sequence[int], parents, T: int,
                               out, lse, stream=None):
    """Verification attention for callers that may not allocate device memory (a host application
    that owns the whole memory pool, or a loop that cannot afford cudaMalloc): no context, no
    workspace -- the scratch is a fixed array inside the library.  Works on the current device;
    calls sharing the device must not overlap on the GPU."""
    kl = _i32_array(kv_len)
    _chk(lib().sparrow_verify_attn_static(ctypes.byref(layout), _ptr(q), _ptr(k_cache), _ptr(v_cache), kl,
                                          _ptr(parents), T, _ptr(out), _ptr(lse), _stream_handle(stream)),
         "sparrow_verify_attn_static")


class VerifyCall(ctypes.Structure):
    _fields_ = [("q", ctypes.c_void_p), ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
                ("kv_len", ctypes.c_void_p), ("parents", ctypes.c_void_p), ("T", ctypes.c_int32),
                ("out", ctypes.c_void_p), ("lse", ctypes.c_void_p)]


class VerifyBatch:
    """A prepared array of sparrow_verify_call records (keeps the host kv_len arrays alive)."""

    def __init__(self, calls):
        """calls: iterable of (q, k_cache, v_cache, kv_len, parents, T, out, lse)."""
        calls = list(calls)
        self._keep = []
        self.array = (VerifyCall * len(calls))()
        for i, (q, k, v, kv_len, parents, T, out, lse) in enumerate(calls):
            kl = _i32_array(kv_len)
            self._keep.append((kl, q, k, v, parents, out, lse))
            self.array[i] = VerifyCall(_ptr(q), _ptr(k), _ptr(v), ctypes.cast(kl, ctypes.c_void_p), _ptr(parents),
                                       T, _ptr(out), _ptr(lse))
        self.n = len(calls)


def sparrow_verify_attn_batch(ctx: Context, batch: VerifyBatch, n_calls: Optional[int] = None, stream=None):
    n = batch.n if n_calls is None else n_calls
    _chk(lib().sparrow_verify_attn_batch(ctx.handle, batch.array, n, _stream_handle(stream)),
         "sparrow_verify_attn_batch")


def sparrow_anchor_attn(ctx: Context, q, k, v, anchor_idx, n_anchor: int, window: int, T: int, out, lse,
                        stream=None):
    _chk(lib().sparrow_anchor_attn(ctx.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(anchor_idx), n_anchor,
                                   window, T, _ptr(out), _ptr(lse), _stream_handle(stream)),
         "sparrow_anchor_attn")


def sparrow_anchor_attn_tree(ctx: Context, q, k, v, anchor_idx, n_anchor: int, window: int, parents, T_tree: int,
                             T_new: int, out, lse, stream=None):
    _chk(lib().sparrow_anchor_attn_tree(ctx.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(anchor_idx), n_anchor,
                                        window, _ptr(parents), T_tree, T_new, _ptr(out), _ptr(lse),
                                        _stream_handle(stream)),
         "sparrow_anchor_attn_tree")


def sparrow_kv_append(ctx: Context, k_new, v_new, k_cache, v_cache, kv_len: Sequence[int], T: int, stream=None):
    _chk(lib().sparrow_kv_append(ctx.handle, _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache),
                                 _i32_array(kv_len), T, _stream_handle(stream)), "sparrow_kv_append")


def sparrow_compact_anchors(ctx: Context, k, v, anchor_idx, n_anchor: int, k_compact, v_compact,
                            compact_capacity: int, dst_row: int = 0, stream=None):
    _chk(lib().sparrow_compact_anchors(ctx.handle, _ptr(k), _ptr(v), _ptr(anchor_idx), n_anchor, _ptr(k_compact),
                                       _ptr(v_compact), compact_capacity, dst_row, _stream_handle(stream)),
         "sparrow_compact_anchors")


def sparrow_accept_greedy(ctx: Context, draft_tokens, parents, target_next, T: int, path_out, n_accept_out,
                          bonus_out, stream=None):
    _chk(lib().sparrow_accept_greedy(ctx.handle, _ptr(draft_tokens), _ptr(parents), _ptr(target_next), T,
                                     _ptr(path_out), _ptr(n_accept_out), _ptr(bonus_out), _stream_handle(stream)),
         "sparrow_accept_greedy")


def sparrow_hsr_fuse(ctx: Context, e, h, w, bias, z, stream=None):
    """z = [e | h] @ w.T (+ bias).  e, h: CUDA bf16 [M, d]; w: CUDA bf16 [d_out, 2d]; bias: CUDA bf16
    [d_out] or None; z: CUDA bf16 [M, d_out]."""
    M, d = e.shape
    d_out = w.shape[0]
    _chk(lib().sparrow_hsr_fuse(ctx.handle, _ptr(e), _ptr(h), _ptr(w), _ptr(bias), M, d, d_out, _ptr(z),
                                _stream_handle(stream)),
         "sparrow_hsr_fuse")


def sparrow_accept_sample(ctx: Context, draft_tokens, parents, p_target, p_draft, u_node, u_bonus, vocab: int, T: int,
                          path_out, n_accept_out, bonus_out, stream=None):
    """Temperature-1 acceptance.  p_target / p_draft: CUDA fp32 [B, T+1, vocab]; u_node: CUDA int32
    [B, T] and u_bonus: CUDA int32 [B, T+1] holding the bit patterns of 32-bit unsigned uniforms."""
    _chk(lib().sparrow_accept_sample(ctx.handle, _ptr(draft_tokens), _ptr(parents), _ptr(p_target), _ptr(p_draft),
                                     _ptr(u_node), _ptr(u_bonus), vocab, T, _ptr(path_out), _ptr(n_accept_out),
                                     _ptr(bonus_out), _stream_handle(stream)), "sparrow_accept_sample")


def sparrow_kv_keep_accepted(ctx: Context, k_cache, v_cache, kv_len: Sequence[int], path, n_accept, T: int,
                             stream=None):
    _chk(lib().sparrow_kv_keep_accepted(ctx.handle, _ptr(k_cache), _ptr(v_cache), _i32_array(kv_len), _ptr(path),
                                        _ptr(n_accept), T, _stream_handle(stream)), "sparrow_kv_keep_accepted")


def sparrow_verify_step_host(ctx: Context, q_host, k_new_host, v_new_host, k_cache, v_cache,
                             kv_len: Sequence[int], parents_host, T: int, out_host, lse_host, stream=None):
    """Host tensors (ideally pinned) in and out; the caches stay on the device."""
    kl = _i32_array(kv_len)
    _chk(lib().sparrow_verify_step_host(ctx.handle, _ptr(q_host), _ptr(k_new_host), _ptr(v_new_host),
                                        _ptr(k_cache), _ptr(v_cache), kl, _ptr(parents_host), T,
                                        _ptr(out_host), _ptr(lse_host), _stream_handle(stream)),
         "sparrow_verify_step_host")


def sparrow_build_ancestor_masks(parents: Sequence[int]):
    T = len(parents)
    par = _i32_array(parents)
    masks = (ctypes.c_uint64 * max(T, 1))()
    _chk(lib().sparrow_build_ancestor_masks(par, T, masks), "sparrow_build_ancestor_masks")
    return [int(masks[i]) for i in range(T)]


def sparrow_build_anchor_idx(seq_len: int, vis_spans, window: int, T: int):
    flat = [int(x) for s in vis_spans for x in s]
    spans = _i32_array(flat) if flat else None
    idx = (ctypes.c_int32 * (max(seq_len, 0) + max(T, 0) + 1))()
    n = ctypes.c_int32(0)
    _chk(lib().sparrow_build_anchor_idx(seq_len, spans, len(flat) // 2, window, T, idx, ctypes.byref(n)),
         "sparrow_build_anchor_idx")
    return [int(idx[i]) for i in range(n.value)]


def sparrow_debug_ancestor_masks_device(ctx: Context, parents_dev: torch.Tensor, T: int, stream=None):
    masks = torch.zeros(T, dtype=torch.int64, device=parents_dev.device)
    _chk(lib().sparrow_debug_ancestor_masks_device(ctx.handle, _ptr(parents_dev), T, _ptr(masks),
                                                   _stream_handle(stream)),
         "sparrow_debug_ancestor_masks_device")
    return masks


def sparrow_debug_wait_counter(ctx: Context, ahead: int, stream=None):
    _chk(lib().sparrow_debug_wait_counter(ctx.handle, ahead, _stream_handle(stream)), "sparrow_debug_wait_counter")


def sparrow_debug_early_trigger_copy(ctx: Context, src, dst, nbytes: int, delay_us: int, stream=None):
    _chk(lib().sparrow_debug_early_trigger_copy(ctx.handle, _ptr(src), _ptr(dst), nbytes, delay_us,
                                                _stream_handle(stream)), "sparrow_debug_early_trigger_copy")


def sparrow_plan_splits(n_sm: int, n_kv_heads: int, n_keys: Sequence[int], T: int, gqa_group: int = 7):
    nk = _i32_array(n_keys)
    splits = (ctypes.c_int32 * len(n_keys))()
    n_items = ctypes.c_int32(0)
    _chk(lib().sparrow_plan_splits(n_sm, len(n_keys), n_kv_heads, gqa_group, nk, T, splits, ctypes.byref(n_items)),
         "sparrow_plan_splits")
    return [int(x) for x in splits], int(n_items.value)


def sparrow_plan_piece_range(n_keys: int, n_splits: int, piece: int):
    b, e = ctypes.c_int32(0), ctypes.c_int32(0)
    _chk(lib().sparrow_plan_piece_range(n_keys, n_splits, piece, ctypes.byref(b), ctypes.byref(e)),
         "sparrow_plan_piece_range")
    return b.value, e.value


def sparrow_status_string(status: int) -> str:
    return lib().sparrow_status_string(status).decode()
