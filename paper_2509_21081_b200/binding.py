"""ctypes binding of the C-ABI library (argument marshalling only).

Every function here has the name of the C entry point it forwards to and does
no arithmetic of its own.  torch tensors are used as device buffers: the
binding passes ``tensor.data_ptr()`` and the current CUDA stream.  There is no
CPU fallback: if the shared library is missing the import of this module
raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtyphoon_mla.so")

MODE_AUTO, MODE_ABSORB, MODE_HYBRID, MODE_NAIVE = 0, 1, 2, 3
MODE_NAMES = {0: "auto", 1: "absorb", 2: "hybrid", 3: "naive"}
COST_NAIVE, COST_ABSORB, COST_TYPHOON = 0, 1, 2
OK = 0


class Dims(C.Structure):
    _fields_ = [("num_heads", C.c_int32), ("d_nope", C.c_int32), ("d_rope", C.c_int32),
                ("d_v", C.c_int32), ("kv_lora_rank", C.c_int32)]


class TyphoonMLAError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib.typhoon_mla_status_string(status).decode()
        extra = ""
        if status == 5:
            extra = f" (cudaError {_lib.typhoon_mla_last_cuda_error()})"
        super().__init__(f"{where}: {msg}{extra}")


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} not found: build it with `python -m paper_2509_21081_b200.build` "
            "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, f32, f64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_double, C.c_size_t
    lib.typhoon_mla_status_string.restype = C.c_char_p
    lib.typhoon_mla_status_string.argtypes = [C.c_int]
    lib.typhoon_mla_prepare_shared.restype = C.c_int
    lib.typhoon_mla_prepare_shared.argtypes = [C.POINTER(Dims), vp, vp, i64, i64, i64, vp, vp, vp, C.POINTER(vp)]
    lib.typhoon_mla_prepare_shared_fp8.restype = C.c_int
    lib.typhoon_mla_prepare_shared_fp8.argtypes = [C.POINTER(Dims), vp, vp, i64, i64, i64, vp, vp, vp, C.POINTER(vp)]
    lib.typhoon_mla_free.restype = C.c_int
    lib.typhoon_mla_free.argtypes = [vp]
    lib.typhoon_mla_workspace_bytes.restype = sz
    lib.typhoon_mla_workspace_bytes.argtypes = [vp, i32, i32, i32, i32]
    lib.typhoon_mla_decode.restype = C.c_int
    lib.typhoon_mla_decode.argtypes = [vp, vp, vp, i32, vp, vp, i64, i64, i32, i32, vp, i32, vp, f32, i32, vp, vp,
                                       vp, sz, vp]
    lib.typhoon_mla_tree_workspace_bytes.restype = sz
    lib.typhoon_mla_decode_partial.restype = C.c_int
    lib.typhoon_mla_decode_partial.argtypes = list(lib.typhoon_mla_decode.argtypes)
    lib.typhoon_mla_combine_partials.restype = C.c_int
    lib.typhoon_mla_combine_partials.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp]
    lib.typhoon_mla_tree_workspace_bytes.argtypes = [vp, i32, i32, i32, i32]
    lib.typhoon_mla_decode_tree.restype = C.c_int
    lib.typhoon_mla_decode_tree.argtypes = [vp, i32, vp, vp, i32, vp, vp, i64, i64, i32, i32, vp, i32, vp, f32, vp, vp,
                                            vp, sz, vp]
    lib.typhoon_mla_host_staging_bytes.restype = sz
    lib.typhoon_mla_host_staging_bytes.argtypes = [vp, i32, i32]
    lib.typhoon_mla_decode_host.restype = C.c_int
    lib.typhoon_mla_decode_host.argtypes = [vp, vp, vp, i32, vp, vp, i64, i64, i32, i32, vp, i32, vp, f32, i32, vp,
                                            vp, sz, vp, sz, vp]
    lib.typhoon_mla_choose_mode.restype = C.c_int
    lib.typhoon_mla_choose_mode.argtypes = [vp, i32, i64]
    lib.typhoon_mla_choose_mode_for.restype = C.c_int
    lib.typhoon_mla_choose_mode_for.argtypes = [C.POINTER(Dims), i64, i32, i64]
    lib.typhoon_mla_set_hw_model.restype = C.c_int
    lib.typhoon_mla_set_hw_model.argtypes = [f64, f64, f64]
    lib.typhoon_mla_set_absorb_efficiency.restype = C.c_int
    lib.typhoon_mla_set_absorb_efficiency.argtypes = [f64]
    lib.typhoon_mla_batch_threshold.restype = f64
    lib.typhoon_mla_batch_threshold.argtypes = [C.POINTER(Dims), i32, f64, f64]
    lib.typhoon_mla_cost_model.restype = C.c_int
    lib.typhoon_mla_cost_model.argtypes = [C.POINTER(Dims), i32, i64, i64, i64, i64, C.POINTER(i64), C.POINTER(i64)]
    lib.typhoon_mla_naive_plan.restype = C.c_int
    lib.typhoon_mla_naive_plan.argtypes = [i32, i32, i64, i32, i32, C.POINTER(i32), C.POINTER(i32), C.POINTER(i32), C.POINTER(i32)]
    lib.typhoon_mla_shared_view.restype = C.c_int
    lib.typhoon_mla_shared_view.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(i64), C.POINTER(i64),
                                            C.POINTER(i64)]
    lib.typhoon_mla_shared_export.restype = C.c_int
    lib.typhoon_mla_shared_export.argtypes = [vp, vp, vp, vp]
    lib.typhoon_mla_shared_export_fp8.restype = C.c_int
    lib.typhoon_mla_shared_export_fp8.argtypes = [vp, vp, vp, vp, vp]
    lib.typhoon_mla_set_kernel_path.restype = C.c_int
    lib.typhoon_mla_set_kernel_path.argtypes = [i32]
    lib.typhoon_mla_order_by_length.restype = C.c_int
    lib.typhoon_mla_order_by_length.argtypes = [vp, i32, vp, vp]
    lib.typhoon_mla_expand_query_rows.restype = C.c_int
    lib.typhoon_mla_expand_query_rows.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp]
    lib.typhoon_mla_set_naive_schedule.restype = C.c_int
    lib.typhoon_mla_set_naive_schedule.argtypes = [i32]
    lib.typhoon_mla_set_programmatic_launch.restype = C.c_int
    lib.typhoon_mla_set_programmatic_launch.argtypes = [i32]
    lib.typhoon_mla_set_overlap.restype = C.c_int
    lib.typhoon_mla_set_overlap.argtypes = [i32]
    lib.typhoon_mla_check_status.restype = C.c_int
    lib.typhoon_mla_check_status.argtypes = [vp, vp, C.POINTER(i32), i32]
    lib.typhoon_mla_test_wait_expiry.restype = C.c_int
    lib.typhoon_mla_test_wait_expiry.argtypes = [vp, i64, i32, vp]
    lib.typhoon_mla_set_stacked_absorb.restype = C.c_int
    lib.typhoon_mla_set_stacked_absorb.argtypes = [i32]
    lib.typhoon_mla_naive_shared_noalloc.restype = C.c_int
    lib.typhoon_mla_naive_shared_noalloc.argtypes = [vp, vp, vp, i32, f32, vp, vp, vp]
    lib.typhoon_mla_profile_begin.restype = C.c_int
    lib.typhoon_mla_profile_begin.argtypes = [i32, i32]
    lib.typhoon_mla_profile_end.restype = C.c_int
    lib.typhoon_mla_profile_end.argtypes = [C.POINTER(f64), C.POINTER(i32)]
    lib.typhoon_mla_last_launch_count.restype = C.c_int
    lib.typhoon_mla_last_cuda_error.restype = C.c_int
    return lib


_lib = _load()


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status: int, where: str):
    if status != OK:
        raise TyphoonMLAError(status, where)


def make_dims(H: int, d_nope=128, d_rope=64, d_v=128, kv_lora_rank=512) -> Dims:
    return Dims(H, d_nope, d_rope, d_v, kv_lora_rank)


class SharedPrefix:
    """Owner of the handle returned by typhoon_mla_prepare_shared."""

    def __init__(self, handle, dims: Dims, keepalive):
        self.handle = handle
        self.dims = dims
        self._keepalive = keepalive

    def free(self):
        if self.handle:
            typhoon_mla_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def typhoon_mla_prepare_shared(dims: Dims, ckv_shared: torch.Tensor, kpe_shared: torch.Tensor,
                               w_uk: torch.Tensor, w_uv: torch.Tensor) -> SharedPrefix:
    Ls = ckv_shared.shape[0]
    h = C.c_void_p()
    ld_ckv = ckv_shared.stride(0) if Ls > 0 else 512
    ld_kpe = kpe_shared.stride(0) if Ls > 0 else 64
    st = _lib.typhoon_mla_prepare_shared(C.byref(dims), _ptr(ckv_shared), _ptr(kpe_shared), Ls, ld_ckv, ld_kpe,
                                         _ptr(w_uk), _ptr(w_uv), _stream(), C.byref(h))
    _check(st, "typhoon_mla_prepare_shared")
    return SharedPrefix(h, dims, (w_uk, w_uv))


def typhoon_mla_prepare_shared_fp8(dims: Dims, ckv_shared: torch.Tensor, kpe_shared: torch.Tensor,
                                   w_uk: torch.Tensor, w_uv: torch.Tensor) -> SharedPrefix:
    """The same with the expanded K_nope / V stored as E4M3 codes (one power-of-two scale per head and tensor)."""
    Ls = ckv_shared.shape[0]
    h = C.c_void_p()
    ld_ckv = ckv_shared.stride(0) if Ls > 0 else 512
    ld_kpe = kpe_shared.stride(0) if Ls > 0 else 64
    st = _lib.typhoon_mla_prepare_shared_fp8(C.byref(dims), _ptr(ckv_shared), _ptr(kpe_shared), Ls, ld_ckv, ld_kpe,
                                             _ptr(w_uk), _ptr(w_uv), _stream(), C.byref(h))
    _check(st, "typhoon_mla_prepare_shared_fp8")
    return SharedPrefix(h, dims, (w_uk, w_uv))


def typhoon_mla_free(handle) -> None:
    _check(_lib.typhoon_mla_free(handle), "typhoon_mla_free")


def typhoon_mla_workspace_bytes(shared: SharedPrefix, B: int, max_pages: int, page_size: int,
                                mode: int = MODE_AUTO) -> int:
    return int(_lib.typhoon_mla_workspace_bytes(shared.handle, B, max_pages, page_size, mode))


def _num_pages(num_pages: Optional[int], ckv_pages) -> int:
    """Physical pages of the cache: the leading extent of the page array unless given."""
    if num_pages is not None:
        return int(num_pages)
    return 0 if ckv_pages is None else int(ckv_pages.shape[0])


def typhoon_mla_decode(shared: SharedPrefix, q_nope, q_pe, ckv_pages, kpe_pages, page_size, block_table,
                       seq_lens, softmax_scale, out, workspace, mode=MODE_AUTO, lse_out=None,
                       max_pages: Optional[int] = None, ckv_token_stride: Optional[int] = None,
                       kpe_token_stride: Optional[int] = None, num_pages: Optional[int] = None) -> None:
    B = q_nope.shape[0]
    if max_pages is None:
        max_pages = 0 if block_table is None else block_table.shape[1]
    if ckv_token_stride is None:
        ckv_token_stride = 512 if ckv_pages is None else ckv_pages.stride(-2)
    if kpe_token_stride is None:
        kpe_token_stride = 64 if kpe_pages is None else kpe_pages.stride(-2)
    st = _lib.typhoon_mla_decode(shared.handle, _ptr(q_nope), _ptr(q_pe), B, _ptr(ckv_pages), _ptr(kpe_pages),
                                 ckv_token_stride, kpe_token_stride, page_size, _num_pages(num_pages, ckv_pages),
                                 _ptr(block_table), max_pages,
                                 _ptr(seq_lens), softmax_scale, mode, _ptr(out), _ptr(lse_out),
                                 _ptr(workspace), workspace.numel() * workspace.element_size(), _stream())
    _check(st, "typhoon_mla_decode")


def typhoon_mla_decode_partial(shared: SharedPrefix, q_nope, q_pe, ckv_pages, kpe_pages, page_size, block_table,
                               seq_lens, softmax_scale, out_partial, lse_partial, workspace, mode=MODE_AUTO,
                               max_pages: Optional[int] = None, ckv_token_stride: Optional[int] = None,
                               kpe_token_stride: Optional[int] = None, num_pages: Optional[int] = None) -> None:
    """This device's share of a sharded context: fp32 out_partial [B, H, 128] and lse_partial [B, H]."""
    B = q_nope.shape[0]
    if max_pages is None:
        max_pages = 0 if block_table is None else block_table.shape[1]
    if ckv_token_stride is None:
        ckv_token_stride = 512 if ckv_pages is None else ckv_pages.stride(-2)
    if kpe_token_stride is None:
        kpe_token_stride = 64 if kpe_pages is None else kpe_pages.stride(-2)
    st = _lib.typhoon_mla_decode_partial(shared.handle, _ptr(q_nope), _ptr(q_pe), B, _ptr(ckv_pages), _ptr(kpe_pages),
                                         ckv_token_stride, kpe_token_stride, page_size, _num_pages(num_pages, ckv_pages),
                                         _ptr(block_table), max_pages,
                                         _ptr(seq_lens), softmax_scale, mode, _ptr(out_partial), _ptr(lse_partial),
                                         _ptr(workspace), workspace.numel() * workspace.element_size(), _stream())
    _check(st, "typhoon_mla_decode_partial")


def typhoon_mla_combine_partials(o_parts, lse_parts, out, lse_out=None) -> None:
    """o_parts fp32 [n, B, H, 128], lse_parts fp32 [n, B, H] -> out bf16 [B, H, 128] (+ lse_out fp32 [B, H])."""
    n, B, H = lse_parts.shape
    st = _lib.typhoon_mla_combine_partials(_ptr(o_parts), _ptr(lse_parts), n, B, H, _ptr(out), _ptr(lse_out), _stream())
    _check(st, "typhoon_mla_combine_partials")


class PrefixLevel(C.Structure):
    """typhoon_mla_prefix_level_t"""
    _fields_ = [("prefixes", C.POINTER(C.c_void_p)), ("group_begin", C.POINTER(C.c_int32)), ("n_groups", C.c_int32)]


def _marshal_levels(levels):
    """levels: list of (prefixes, group_begin) with prefixes a list of SharedPrefix or None.
    Returns (array of PrefixLevel, keepalive)."""
    arr = (PrefixLevel * len(levels))()
    keep = []
    for i, (prefixes, group_begin) in enumerate(levels):
        if len(group_begin) != len(prefixes) + 1:
            raise ValueError("group_begin needs one more entry than prefixes")
        hp = (C.c_void_p * len(prefixes))(*[None if p is None else p.handle.value for p in prefixes])
        gb = (C.c_int32 * len(group_begin))(*group_begin)
        keep += [hp, gb]
        arr[i] = PrefixLevel(C.cast(hp, C.POINTER(C.c_void_p)), C.cast(gb, C.POINTER(C.c_int32)), len(prefixes))
    return arr, keep


def typhoon_mla_tree_workspace_bytes(levels, B: int, max_pages: int, page_size: int) -> int:
    arr, keep = _marshal_levels(levels)
    return int(_lib.typhoon_mla_tree_workspace_bytes(C.cast(arr, C.c_void_p), len(levels), B, max_pages, page_size))


def typhoon_mla_decode_tree(levels, q_nope, q_pe, ckv_pages, kpe_pages, page_size, block_table, seq_lens,
                            softmax_scale, out, workspace, lse_out=None, num_pages: Optional[int] = None) -> None:
    arr, keep = _marshal_levels(levels)
    B = q_nope.shape[0]
    max_pages = 0 if block_table is None else block_table.shape[1]
    st = _lib.typhoon_mla_decode_tree(
        C.cast(arr, C.c_void_p), len(levels), _ptr(q_nope), _ptr(q_pe), B, _ptr(ckv_pages), _ptr(kpe_pages),
        512 if ckv_pages is None else ckv_pages.stride(-2), 64 if kpe_pages is None else kpe_pages.stride(-2),
        page_size, _num_pages(num_pages, ckv_pages), _ptr(block_table), max_pages, _ptr(seq_lens), softmax_scale,
        _ptr(out), _ptr(lse_out),
        _ptr(workspace), workspace.numel() * workspace.element_size(), _stream())
    _check(st, "typhoon_mla_decode_tree")


def typhoon_mla_host_staging_bytes(shared: SharedPrefix, B: int, max_pages: int) -> int:
    return int(_lib.typhoon_mla_host_staging_bytes(shared.handle, B, max_pages))


def typhoon_mla_decode_host(shared: SharedPrefix, q_nope_host, q_pe_host, ckv_pages, kpe_pages, page_size,
                            block_table_host, seq_lens_host, softmax_scale, out_host, staging, workspace,
                            mode=MODE_AUTO, num_pages: Optional[int] = None) -> None:
    B = q_nope_host.shape[0]
    max_pages = 0 if block_table_host is None else block_table_host.shape[1]
    st = _lib.typhoon_mla_decode_host(
        shared.handle, _ptr(q_nope_host), _ptr(q_pe_host), B, _ptr(ckv_pages), _ptr(kpe_pages),
        512 if ckv_pages is None else ckv_pages.stride(-2), 64 if kpe_pages is None else kpe_pages.stride(-2),
        page_size, _num_pages(num_pages, ckv_pages), _ptr(block_table_host), max_pages, _ptr(seq_lens_host),
        softmax_scale, mode, _ptr(out_host),
        _ptr(staging), staging.numel() * staging.element_size(),
        _ptr(workspace), workspace.numel() * workspace.element_size(), _stream())
    _check(st, "typhoon_mla_decode_host")


def typhoon_mla_choose_mode(shared: SharedPrefix, B: int, total_suffix_tokens: int = -1) -> int:
    return int(_lib.typhoon_mla_choose_mode(shared.handle, B, total_suffix_tokens))


def typhoon_mla_choose_mode_for(dims: Dims, Ls: int, B: int, total_suffix_tokens: int = -1) -> int:
    return int(_lib.typhoon_mla_choose_mode_for(C.byref(dims), Ls, B, total_suffix_tokens))


def typhoon_mla_set_hw_model(tensor_flops: float, hbm_bytes_per_s: float, hybrid_fixed_s: float) -> None:
    _check(_lib.typhoon_mla_set_hw_model(tensor_flops, hbm_bytes_per_s, hybrid_fixed_s), "typhoon_mla_set_hw_model")


def typhoon_mla_batch_threshold(dims: Dims, S_q: int, T: float, M: float) -> float:
    return float(_lib.typhoon_mla_batch_threshold(C.byref(dims), S_q, T, M))


def typhoon_mla_cost_model(dims: Dims, kind: int, B: int, S_q: int, L_s: int, L_n: int):
    m, w = C.c_int64(), C.c_int64()
    _check(_lib.typhoon_mla_cost_model(C.byref(dims), kind, B, S_q, L_s, L_n, C.byref(m), C.byref(w)),
           "typhoon_mla_cost_model")
    return m.value, w.value


def typhoon_mla_naive_plan(num_heads: int, B: int, L_s: int, schedule: int = 0, num_sms: int = 0):
    """(tile_tokens, n_ranges, row_groups, n_slots) of the shared-prefix kernel's work decomposition."""
    t, r, g, sl = C.c_int32(), C.c_int32(), C.c_int32(), C.c_int32()
    _check(_lib.typhoon_mla_naive_plan(num_heads, B, L_s, schedule, num_sms, C.byref(t), C.byref(r), C.byref(g), C.byref(sl)),
           "typhoon_mla_naive_plan")
    return t.value, r.value, g.value, sl.value


def typhoon_mla_shared_view(shared: SharedPrefix):
    """(Ls, Ls_padded, owned_bytes) of the handle."""
    k, v = C.c_void_p(), C.c_void_p()
    Ls, Lp, ob = C.c_int64(), C.c_int64(), C.c_int64()
    _check(_lib.typhoon_mla_shared_view(shared.handle, C.byref(k), C.byref(v), C.byref(Ls), C.byref(Lp), C.byref(ob)),
           "typhoon_mla_shared_view")
    return Ls.value, Lp.value, ob.value


def typhoon_mla_shared_export(shared: SharedPrefix):
    """Copies of the expanded caches: k_nope [H, Ls_pad/64, 2, 64, 64], v_t [H, Ls_pad/64, 128, 64]."""
    _, Lp, _ = typhoon_mla_shared_view(shared)
    H = shared.dims.num_heads
    kt = torch.empty(H, Lp // 64, 2, 64, 64, dtype=torch.bfloat16, device="cuda")
    vt = torch.empty(H, Lp // 64, 128, 64, dtype=torch.bfloat16, device="cuda")
    _check(_lib.typhoon_mla_shared_export(shared.handle, _ptr(kt), _ptr(vt), _stream()), "typhoon_mla_shared_export")
    return kt, vt


def typhoon_mla_shared_export_fp8(shared: SharedPrefix):
    """Codes and scales of an 8-bit handle: K codes uint8 [H, Ls_pad, 128], V codes uint8 [H, Ls_pad/64, 128, 64]
    (V^T in 64-token blocks), scales float32 [2, H] (K_nope, V)."""
    _, Lp, _ = typhoon_mla_shared_view(shared)
    H = shared.dims.num_heads
    kc = torch.empty(H, Lp, 128, dtype=torch.uint8, device="cuda")
    vc = torch.empty(H, Lp // 64, 128, 64, dtype=torch.uint8, device="cuda")
    sc = torch.empty(2, H, dtype=torch.float32, device="cuda")
    _check(_lib.typhoon_mla_shared_export_fp8(shared.handle, _ptr(kc), _ptr(vc), _ptr(sc), _stream()),
           "typhoon_mla_shared_export_fp8")
    return kc, vc, sc


def typhoon_mla_last_launch_count() -> int:
    return int(_lib.typhoon_mla_last_launch_count())


KERNEL_NAMES = ("naive_attn", "q_absorb", "absorb_attn", "merge", "w_uv", "combine")


def typhoon_mla_profile_begin(kernel_id: int, max_launches: int) -> None:
    _check(_lib.typhoon_mla_profile_begin(kernel_id, max_launches), "typhoon_mla_profile_begin")


def typhoon_mla_profile_end():
    ms, n = C.c_double(), C.c_int32()
    _check(_lib.typhoon_mla_profile_end(C.byref(ms), C.byref(n)), "typhoon_mla_profile_end")
    return ms.value, n.value


NOALLOC_SCRATCH_BYTES = 32 << 20


def typhoon_mla_naive_shared_noalloc(shared: SharedPrefix, q_nope, q_pe, softmax_scale, out, lse_out=None) -> None:
    """Shared-prefix attention using the library's built-in scratch array: no workspace argument and
    no allocation, for callers that cannot get device memory at call time."""
    st = _lib.typhoon_mla_naive_shared_noalloc(shared.handle, _ptr(q_nope), _ptr(q_pe), q_nope.shape[0],
                                               softmax_scale, _ptr(out), _ptr(lse_out), _stream())
    _check(st, "typhoon_mla_naive_shared_noalloc")


PATH_TCGEN05, PATH_WARP_MMA = 0, 1


def typhoon_mla_set_kernel_path(path: int) -> None:
    _check(_lib.typhoon_mla_set_kernel_path(path), "typhoon_mla_set_kernel_path")


STATUS_WAIT_EXPIRED, STATUS_BAD_PAGE = 0xFF, 0x100


def typhoon_mla_check_status(shared: SharedPrefix, clear: bool = False, raise_on_error: bool = True) -> int:
    """Synchronises the current stream and returns the handle's device status word; raises if it is
    non-zero (a bounded in-kernel wait ran out, or a page id was out of range) unless told not to."""
    v = C.c_int32()
    st = _lib.typhoon_mla_check_status(shared.handle, _stream(), C.byref(v), 1 if clear else 0)
    if raise_on_error or st not in (0, 6):
        _check(st, "typhoon_mla_check_status")
    return v.value


def typhoon_mla_test_wait_expiry(shared: SharedPrefix, deadline_cycles: int, code: int = 0x40) -> None:
    _check(_lib.typhoon_mla_test_wait_expiry(shared.handle, deadline_cycles, code, _stream()),
           "typhoon_mla_test_wait_expiry")


def typhoon_mla_set_stacked_absorb(enable: bool) -> None:
    _check(_lib.typhoon_mla_set_stacked_absorb(1 if enable else 0), "typhoon_mla_set_stacked_absorb")


def typhoon_mla_expand_query_rows(block_table: torch.Tensor, seq_lens: torch.Tensor, S_q: int):
    """(block_table_rows [B*S_q, max_pages], seq_lens_rows [B*S_q]) for S_q query tokens per request."""
    B, max_pages = block_table.shape
    bt = torch.empty(B * S_q, max_pages, dtype=torch.int32, device=block_table.device)
    sl = torch.empty(B * S_q, dtype=torch.int32, device=block_table.device)
    _check(_lib.typhoon_mla_expand_query_rows(_ptr(block_table), _ptr(seq_lens), B, max_pages, S_q, _ptr(bt), _ptr(sl),
                                              _stream()), "typhoon_mla_expand_query_rows")
    return bt, sl


def typhoon_mla_set_naive_schedule(schedule: int) -> None:
    _check(_lib.typhoon_mla_set_naive_schedule(schedule), "typhoon_mla_set_naive_schedule")


def typhoon_mla_set_programmatic_launch(enable: bool) -> None:
    _check(_lib.typhoon_mla_set_programmatic_launch(1 if enable else 0), "typhoon_mla_set_programmatic_launch")


def typhoon_mla_set_overlap(enable: bool) -> None:
    _check(_lib.typhoon_mla_set_overlap(1 if enable else 0), "typhoon_mla_set_overlap")


def typhoon_mla_order_by_length(seq_lens: torch.Tensor) -> torch.Tensor:
    perm = torch.empty_like(seq_lens)
    _check(_lib.typhoon_mla_order_by_length(_ptr(seq_lens), seq_lens.numel(), _ptr(perm), _stream()),
           "typhoon_mla_order_by_length")
    return perm


def typhoon_mla_set_absorb_efficiency(fraction: float) -> None:
    _check(_lib.typhoon_mla_set_absorb_efficiency(fraction), "typhoon_mla_set_absorb_efficiency")
