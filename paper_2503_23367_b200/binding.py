"""ctypes binding of libfastvar.so: same names as the C ABI, argument marshalling only.

Every step of the pruned VAR scale step runs in the CUDA kernels behind the C ABI; torch is used here
for device buffers and streams.  There is no CPU fallback: loading fails loudly when the library has
not been built.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfastvar.so")

FV_OK = 0
STATUS_NAMES = {0: "FV_OK", 1: "FV_ERR_INVALID_ARG", 2: "FV_ERR_BAD_STATE", 3: "FV_ERR_CAPACITY",
                4: "FV_ERR_UNSUPPORTED", 5: "FV_ERR_CUDA", 6: "FV_ERR_TIMEOUT", 7: "FV_ERR_DEVICE_DATA"}

EXPORTS = ["fv_status_string", "fv_k_for", "fv_prune_select_workspace_bytes", "fv_prune_select", "fv_restore",
           "fv_workspace_bytes", "fv_kv_bytes", "fv_cache_bytes", "fv_create", "fv_destroy", "fv_reset",
           "fv_get_state", "fv_set_state", "fv_kv_pointers", "fv_cache_pointer", "fv_prepare_text",
           "fv_device_status", "fv_selftest_expired_wait", "fv_var_step", "fv_gather_ln", "fv_restore_residual", "fv_prune_select_after_restore",
           "fv_prune_select_workspace_layout", "fv_restore_force_fold", "fv_step_fused_selection", "fv_gemm_bf16", "fv_gemm_splitk_workspace_bytes", "fv_gemm_force_path", "fv_attention", "fv_attention_workspace_bytes", "fv_attention_force_ctas",
           "fv_kernel_launches", "fv_profile_enable", "fv_profile_read",
           "fv_prune_select_static", "fv_prune_select_static_capacity",
           "fv_head_workspace_bytes", "fv_head_tokens", "fv_argmax_rows", "fv_residual_accumulate", "fv_next_scale_input",
           "fv_generate_workspace_bytes", "fv_generate", "fv_var_step_host_staging_bytes", "fv_var_step_host", "fv_host_io_flush", "fv_struct_sizes"]


class FvError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: {STATUS_NAMES.get(code, code)}")
        self.code = code


class fv_config(C.Structure):
    _fields_ = [("L", C.c_int32), ("C", C.c_int32), ("H", C.c_int32), ("mlp_ratio", C.c_int32),
                ("cross_len", C.c_int32), ("B_max", C.c_int32), ("n_steps", C.c_int32),
                ("h", C.POINTER(C.c_int32)), ("w", C.POINTER(C.c_int32)),
                ("cache_step", C.c_int32), ("kv_capacity", C.c_int32), ("granularity", C.c_int32),
                ("rope_base", C.c_float), ("interp_mode", C.c_int32), ("resid_dtype", C.c_int32)]


class fv_weights(C.Structure):
    _fields_ = [(n, C.POINTER(C.c_void_p)) for n in
                ("w_qkv", "b_qkv", "w_o", "b_o", "w_fc1", "b_fc1", "w_fc2", "b_fc2", "w_q_x", "w_kv_x", "w_o_x")] + \
               [("mod_dev", C.c_void_p), ("text_dev", C.c_void_p), ("qk_scale_dev", C.c_void_p)]


class fv_generator(C.Structure):
    _fields_ = [("V", C.c_int32), ("d", C.c_int32), ("codebook_dev", C.c_void_p), ("w_head_dev", C.c_void_p),
                ("b_head_dev", C.c_void_p), ("mod_head_dev", C.c_void_p), ("w_in_dev", C.c_void_p), ("b_in_dev", C.c_void_p),
                ("pos_dev", C.POINTER(C.c_void_p)), ("tau", C.c_float)]


_lib = None


def lib() -> C.CDLL:
    """Loads libfastvar.so (once).  Raises if it has not been built: there is no fallback path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2503_23367_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, i32, sz, dbl = C.c_void_p, C.c_int32, C.c_size_t, C.c_double
        L.fv_status_string.restype = C.c_char_p; L.fv_status_string.argtypes = [C.c_int]
        L.fv_k_for.restype = i32; L.fv_k_for.argtypes = [dbl, i32, i32]
        L.fv_prune_select_workspace_bytes.restype = sz; L.fv_prune_select_workspace_bytes.argtypes = [i32, i32, i32]
        L.fv_prune_select.restype = C.c_int
        L.fv_prune_select.argtypes = [vp, i32, i32, i32, i32, dbl, vp, vp, vp, vp, C.POINTER(i32), vp, sz, vp]
        L.fv_restore.restype = C.c_int
        L.fv_restore.argtypes = [vp, i32, i32, vp, vp, i32, i32, i32, i32, i32, vp, vp, i32, vp]
        for f in ("fv_workspace_bytes", "fv_kv_bytes", "fv_cache_bytes"):
            getattr(L, f).restype = sz; getattr(L, f).argtypes = [C.POINTER(fv_config)]
        L.fv_create.restype = C.c_int
        L.fv_create.argtypes = [C.POINTER(fv_config), C.POINTER(fv_weights), vp, vp, vp, C.POINTER(vp)]
        L.fv_destroy.restype = None; L.fv_destroy.argtypes = [vp]
        L.fv_reset.restype = C.c_int; L.fv_reset.argtypes = [vp]
        L.fv_get_state.restype = C.c_int; L.fv_get_state.argtypes = [vp, C.POINTER(i32), C.POINTER(i32)]
        L.fv_set_state.restype = C.c_int; L.fv_set_state.argtypes = [vp, i32, i32]
        L.fv_kv_pointers.restype = C.c_int; L.fv_kv_pointers.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(vp)]
        L.fv_cache_pointer.restype = C.c_int; L.fv_cache_pointer.argtypes = [vp, i32, i32, C.POINTER(vp)]
        L.fv_prepare_text.restype = C.c_int; L.fv_prepare_text.argtypes = [vp, i32, vp]
        L.fv_device_status.restype = C.c_int; L.fv_device_status.argtypes = [vp, C.POINTER(i32), vp]
        L.fv_var_step.restype = C.c_int; L.fv_var_step.argtypes = [vp, vp, i32, i32, dbl, vp, vp, vp, vp]
        L.fv_gather_ln.restype = C.c_int; L.fv_gather_ln.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, i32, vp, vp, vp]
        L.fv_selftest_expired_wait.restype = C.c_int; L.fv_selftest_expired_wait.argtypes = [vp, C.c_uint64, vp]
        L.fv_restore_residual.restype = C.c_int
        L.fv_restore_residual.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, i32, i32, vp, sz, i32, vp]
        L.fv_prune_select_after_restore.restype = C.c_int
        L.fv_prune_select_after_restore.argtypes = [vp, i32, i32, i32, i32, dbl, vp, vp, vp, vp, C.POINTER(i32), vp, sz, vp]
        L.fv_prune_select_workspace_layout.restype = C.c_int
        L.fv_prune_select_workspace_layout.argtypes = [i32, i32, i32, C.POINTER(sz), C.POINTER(i32)]
        L.fv_restore_force_fold.restype = C.c_int; L.fv_restore_force_fold.argtypes = [i32]
        L.fv_step_fused_selection.restype = C.c_int; L.fv_step_fused_selection.argtypes = [i32]
        L.fv_gemm_bf16.restype = C.c_int
        L.fv_gemm_bf16.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, i32, i32, vp, vp, sz, vp]
        L.fv_gemm_splitk_workspace_bytes.restype = sz; L.fv_gemm_splitk_workspace_bytes.argtypes = []
        L.fv_gemm_force_path.restype = C.c_int; L.fv_gemm_force_path.argtypes = [i32]
        L.fv_attention.restype = C.c_int
        L.fv_attention.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, sz, vp]
        L.fv_attention_workspace_bytes.restype = sz; L.fv_attention_workspace_bytes.argtypes = []
        L.fv_attention_force_ctas.restype = C.c_int; L.fv_attention_force_ctas.argtypes = [i32]
        L.fv_prune_select_static_capacity.restype = sz; L.fv_prune_select_static_capacity.argtypes = []
        L.fv_prune_select_static.restype = C.c_int
        L.fv_prune_select_static.argtypes = [vp, i32, i32, i32, i32, dbl, vp, vp, vp, vp, C.POINTER(i32), vp]
        f32 = C.c_float
        L.fv_head_workspace_bytes.restype = sz; L.fv_head_workspace_bytes.argtypes = [i32, i32, i32]
        L.fv_head_tokens.restype = C.c_int
        L.fv_head_tokens.argtypes = [vp, i32, i32, i32, vp, vp, vp, i32, vp, f32, vp, vp, vp, sz, vp, vp]
        L.fv_argmax_rows.restype = C.c_int; L.fv_argmax_rows.argtypes = [vp, vp, f32, i32, i32, vp, vp]
        L.fv_residual_accumulate.restype = C.c_int
        L.fv_residual_accumulate.argtypes = [vp, i32, i32, i32, vp, i32, i32, vp, i32, i32, vp, vp, vp]
        L.fv_next_scale_input.restype = C.c_int
        L.fv_next_scale_input.argtypes = [vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, i32, vp, vp]
        L.fv_generate_workspace_bytes.restype = sz; L.fv_generate_workspace_bytes.argtypes = [vp, C.POINTER(fv_generator)]
        L.fv_generate.restype = C.c_int
        L.fv_generate.argtypes = [vp, C.POINTER(fv_generator), vp, i32, C.POINTER(dbl), C.POINTER(vp), vp, vp, vp, sz, vp]
        L.fv_var_step_host_staging_bytes.restype = sz; L.fv_var_step_host_staging_bytes.argtypes = [C.POINTER(fv_config)]
        L.fv_var_step_host.restype = C.c_int; L.fv_var_step_host.argtypes = [vp, vp, i32, i32, dbl, vp, vp, sz, vp]
        L.fv_host_io_flush.restype = C.c_int; L.fv_host_io_flush.argtypes = [vp, vp]
        L.fv_kernel_launches.restype = C.c_uint64; L.fv_kernel_launches.argtypes = []
        L.fv_profile_enable.restype = C.c_int; L.fv_profile_enable.argtypes = [i32]
        L.fv_profile_read.restype = C.c_int
        L.fv_profile_read.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_uint64), C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.fv_struct_sizes.restype = None; L.fv_struct_sizes.argtypes = [C.POINTER(sz)]
        sizes = (sz * 3)()
        L.fv_struct_sizes(sizes)
        mine = (C.sizeof(fv_config), C.sizeof(fv_weights), C.sizeof(fv_generator))
        if tuple(sizes) != mine:
            raise RuntimeError(f"struct layouts of binding.py {mine} and libfastvar.so {tuple(sizes)} differ: rebuild the library")
        _lib = L
    return _lib


def _ptr(t) -> Optional[int]:
    if t is None or isinstance(t, int):
        return t                      # None, or a raw device address (sub-tensor with its own stride)
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(code: int, where: str) -> None:
    if code != FV_OK:
        raise FvError(code, where)


KERNEL_CLASSES = ("select", "gather_ln", "gemm", "attention", "restore")


def fv_kernel_launches() -> int:
    return int(lib().fv_kernel_launches())


def fv_profile_enable(on: bool) -> None:
    _check(lib().fv_profile_enable(1 if on else 0), "fv_profile_enable")


def fv_profile_read() -> dict:
    """{class: {"ms", "launches", "work", "dram_bytes"}}; work = algorithmic bytes (select, gather_ln, restore)
    or flops; dram_bytes = operand + result bytes the launches have to move to and from HBM once."""
    ms, ln, wk, db = (C.c_double * 5)(), (C.c_uint64 * 5)(), (C.c_double * 5)(), (C.c_double * 5)()
    _check(lib().fv_profile_read(ms, ln, wk, db), "fv_profile_read")
    return {n: {"ms": ms[i], "launches": int(ln[i]), "work": wk[i], "dram_bytes": db[i]} for i, n in enumerate(KERNEL_CLASSES)}


def fv_k_for(keep_ratio: float, h: int, w: int) -> int:
    return lib().fv_k_for(float(keep_ratio), h, w)


def fv_prune_select(x: torch.Tensor, h: int, w: int, keep_ratio: float, want_inv=True, want_score=False,
                    want_near_tie=False, workspace: Optional[torch.Tensor] = None):
    """x fp32 [B, h*w, C] -> dict(idx int32 [B,k], inv, score, near_tie, k)."""
    B, n, Cw = x.shape
    assert x.dtype == torch.float32 and n == h * w
    k = fv_k_for(keep_ratio, h, w)
    dev = x.device
    idx = torch.empty((B, k), dtype=torch.int32, device=dev)
    inv = torch.empty((B, n), dtype=torch.int32, device=dev) if want_inv else None
    score = torch.empty((B, n), dtype=torch.float32, device=dev) if want_score else None
    near = torch.empty((B,), dtype=torch.int32, device=dev) if want_near_tie else None
    need = lib().fv_prune_select_workspace_bytes(B, n, Cw)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    k_out = C.c_int32(0)
    _check(lib().fv_prune_select(_ptr(x), B, h, w, Cw, float(keep_ratio), _ptr(idx), _ptr(inv), _ptr(score), _ptr(near),
                                 C.byref(k_out), _ptr(workspace), workspace.numel(), _stream()), "fv_prune_select")
    assert k_out.value == k
    return {"idx": idx, "inv": inv, "score": score, "near_tie": near, "k": k}


def fv_prune_select_static(x: torch.Tensor, h: int, w: int, keep_ratio: float, out: dict) -> int:
    """Selection without a caller workspace, for hosts that cannot allocate: the scratch is a fixed array
    inside the library (see fv_prune_select_static_capacity).  `out` holds the caller's own pre-made
    output tensors: "idx" int32 [B,k] (required), optional "inv" int32 [B,n], "score" fp32 [B,n],
    "near_tie" int32 [B].  Nothing is allocated here or in the library.  Returns k."""
    B, n, Cw = x.shape
    k_out = C.c_int32(0)
    _check(lib().fv_prune_select_static(_ptr(x), B, h, w, Cw, float(keep_ratio), _ptr(out["idx"]), _ptr(out.get("inv")),
                                        _ptr(out.get("score")), _ptr(out.get("near_tie")), C.byref(k_out), _stream()),
           "fv_prune_select_static")
    return k_out.value


def fv_restore(cache_prev: torch.Tensor, hc: int, wc: int, pivots: torch.Tensor, idx: torch.Tensor, h: int, w: int,
               out: Optional[torch.Tensor] = None, interp_mode: int = 0) -> torch.Tensor:
    """cache_prev bf16 [B,hc*wc,C], pivots bf16 [B,k,C], idx int32 [B,k] -> bf16 [B,h*w,C].  interp_mode 0 nearest, 1 bilinear."""
    B, k, Cw = pivots.shape
    if out is None:
        out = torch.empty((B, h * w, Cw), dtype=torch.bfloat16, device=pivots.device)
    inv = torch.empty((B, h * w), dtype=torch.int32, device=pivots.device)
    _check(lib().fv_restore(_ptr(cache_prev), hc, wc, _ptr(pivots), _ptr(idx), B, k, h, w, Cw, _ptr(out), _ptr(inv),
                            int(interp_mode), _stream()), "fv_restore")
    return out


def fv_gather_ln(x: torch.Tensor, idx: Optional[torch.Tensor], sigma: Optional[torch.Tensor],
                 beta: Optional[torch.Tensor], mod_stride: int = 0, status: Optional[torch.Tensor] = None) -> torch.Tensor:
    B, n, Cw = x.shape
    k = n if idx is None else idx.shape[1]
    out = torch.empty((B, k, Cw), dtype=torch.bfloat16, device=x.device)
    _check(lib().fv_gather_ln(_ptr(x), _ptr(idx), B, n, k, Cw, _ptr(sigma), _ptr(beta), mod_stride, _ptr(out), _ptr(status), _stream()),
           "fv_gather_ln")
    return out


def fv_restore_residual(x: torch.Tensor, y: torch.Tensor, cache: torch.Tensor, inv: torch.Tensor,
                        gamma: Optional[torch.Tensor], mod_stride: int, h: int, w: int, hc: int, wc: int, interp_mode: int = 0,
                        colsum_ws: Optional[torch.Tensor] = None, part: int = 0) -> None:
    """colsum_ws: uint8 selection workspace that receives the column sums of the updated map, or None."""
    B, n, Cw = x.shape
    k = y.shape[1]
    _check(lib().fv_restore_residual(_ptr(x), _ptr(y), _ptr(cache), _ptr(inv), _ptr(gamma), mod_stride, B, k, h, w, hc, wc,
                                     Cw, int(interp_mode), _ptr(colsum_ws), 0 if colsum_ws is None else colsum_ws.numel(),
                                     int(part), _stream()), "fv_restore_residual")


def fv_prune_select_workspace(B: int, n: int, Cw: int, device) -> torch.Tensor:
    return torch.empty(lib().fv_prune_select_workspace_bytes(B, n, Cw), dtype=torch.uint8, device=device)


def fv_colsum_partials(workspace: torch.Tensor, B: int, n: int, Cw: int) -> torch.Tensor:
    """fp32 view [B, partials, C] of the column sums a restoration left in a selection workspace."""
    off, cnt = C.c_size_t(), C.c_int32()
    _check(lib().fv_prune_select_workspace_layout(B, n, Cw, C.byref(off), C.byref(cnt)), "fv_prune_select_workspace_layout")
    return workspace[off.value: off.value + 4 * B * cnt.value * Cw].view(torch.float32).view(B, cnt.value, Cw)


def fv_prune_select_after_restore(x: torch.Tensor, h: int, w: int, keep_ratio: float, workspace: torch.Tensor,
                                  want_score: bool = False, want_near_tie: bool = False):
    """fv_prune_select of a map whose column sums fv_restore_residual left in `workspace`."""
    B, n, Cw = x.shape
    k = fv_k_for(keep_ratio, h, w)
    idx = torch.empty((B, k), dtype=torch.int32, device=x.device)
    inv = torch.empty((B, n), dtype=torch.int32, device=x.device)
    score = torch.empty((B, n), dtype=torch.float32, device=x.device) if want_score else None
    near = torch.empty((B,), dtype=torch.int32, device=x.device) if want_near_tie else None
    k_out = C.c_int32(0)
    _check(lib().fv_prune_select_after_restore(_ptr(x), B, h, w, Cw, float(keep_ratio), _ptr(idx), _ptr(inv), _ptr(score), _ptr(near),
                                               C.byref(k_out), _ptr(workspace), workspace.numel(), _stream()),
           "fv_prune_select_after_restore")
    return {"idx": idx, "inv": inv, "score": score, "near_tie": near, "k": k}


def fv_restore_force_fold(mode: int) -> None:
    _check(lib().fv_restore_force_fold(int(mode)), "fv_restore_force_fold")


def fv_gemm_bf16(a: torch.Tensor, w: torch.Tensor, bias: Optional[torch.Tensor], epilogue: int = 0,
                 out: Optional[torch.Tensor] = None, aux: Optional[torch.Tensor] = None,
                 gamma: Optional[torch.Tensor] = None, mod_stride: int = 0, rows_per_image: int = 0,
                 status: Optional[torch.Tensor] = None, splitk_ws: Optional[torch.Tensor] = None) -> torch.Tensor:
    """splitk_ws: uint8 scratch of fv_gemm_splitk_workspace_bytes() bytes, first 4096 zero, or None (no K split)."""
    M, K = a.shape
    N = w.shape[0]
    assert w.shape[1] == K and a.dtype == torch.bfloat16 and w.dtype == torch.bfloat16
    if out is None:
        assert epilogue in (0, 1)
        out = torch.empty((M, N), dtype=torch.bfloat16, device=a.device)
    _check(lib().fv_gemm_bf16(_ptr(a), _ptr(w), _ptr(bias), M, N, K, epilogue, _ptr(out), _ptr(aux), _ptr(gamma),
                              mod_stride, rows_per_image, _ptr(status), _ptr(splitk_ws),
                              0 if splitk_ws is None else splitk_ws.numel(), _stream()), "fv_gemm_bf16")
    return out


def fv_attention_workspace(device) -> torch.Tensor:
    """Zeroed scratch for fv_attention's split over the SMs (its arrival counters must start at zero)."""
    return torch.zeros(lib().fv_attention_workspace_bytes(), dtype=torch.uint8, device=device)


def fv_attention(q: torch.Tensor, k_cache: torch.Tensor, vt_cache: torch.Tensor, B: int, rows: int, H: int, kv_len: int,
                 status: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """q bf16 [B*rows, C]; k_cache bf16 [B, cap, C]; vt_cache bf16 [B, C, cap] -> bf16 [B*rows, C].
    workspace: fv_attention_workspace(...) to cut the work into one piece per SM, or None."""
    Cw = q.shape[1]
    cap = k_cache.shape[1]
    out = torch.empty_like(q)
    _check(lib().fv_attention(_ptr(q), _ptr(k_cache), _ptr(vt_cache), B, rows, H, Cw, kv_len, cap, _ptr(out), _ptr(status),
                              _ptr(workspace), 0 if workspace is None else workspace.numel(), _stream()), "fv_attention")
    return out


def fv_argmax_rows(logits: torch.Tensor, noise: Optional[torch.Tensor] = None, tau: float = 1.0) -> torch.Tensor:
    rows, V = logits.shape
    ids = torch.empty(rows, dtype=torch.int32, device=logits.device)
    _check(lib().fv_argmax_rows(_ptr(logits), _ptr(noise), float(tau), rows, V, _ptr(ids), _stream()), "fv_argmax_rows")
    return ids


def fv_head_tokens(y: torch.Tensor, mod_head: torch.Tensor, w_head: torch.Tensor, b_head: Optional[torch.Tensor],
                   noise: Optional[torch.Tensor] = None, tau: float = 1.0, want_logits: bool = False,
                   status: Optional[torch.Tensor] = None):
    """y fp32 [B, n, C]; returns ids int32 [B, n] (and the fp32 logits [B*n, V] when asked)."""
    B, n, Cw = y.shape
    V = w_head.shape[0]
    ws_bytes = lib().fv_head_workspace_bytes(B * n, Cw, V)
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device=y.device)
    wsp = (ws.data_ptr() + 255) // 256 * 256
    ids = torch.empty((B, n), dtype=torch.int32, device=y.device)
    logits = torch.empty((B * n, V), dtype=torch.float32, device=y.device) if want_logits else None
    _check(lib().fv_head_tokens(_ptr(y), B, n, Cw, _ptr(mod_head), _ptr(w_head), _ptr(b_head), V, _ptr(noise), float(tau),
                                _ptr(ids), _ptr(logits), wsp, ws_bytes, _ptr(status), _stream()), "fv_head_tokens")
    return (ids, logits) if want_logits else ids


def fv_residual_accumulate(ids: torch.Tensor, h: int, w: int, codebook: torch.Tensor, r_prev: Optional[torch.Tensor] = None,
                           hp: int = 0, wp: int = 0, status: Optional[torch.Tensor] = None) -> torch.Tensor:
    B = ids.shape[0]
    V, d = codebook.shape
    out = torch.empty((B, h * w, d), dtype=torch.float32, device=ids.device)
    _check(lib().fv_residual_accumulate(_ptr(ids), B, h, w, _ptr(codebook), V, d, _ptr(r_prev), hp, wp, _ptr(out), _ptr(status),
                                        _stream()), "fv_residual_accumulate")
    return out


def fv_next_scale_input(r: torch.Tensor, h: int, w: int, h2: int, w2: int, w_in: torch.Tensor, b_in: Optional[torch.Tensor],
                        pos: Optional[torch.Tensor]) -> torch.Tensor:
    B, _, d = r.shape
    Cw = w_in.shape[0]
    out = torch.empty((B, h2 * w2, Cw), dtype=torch.float32, device=r.device)
    _check(lib().fv_next_scale_input(_ptr(r), B, h, w, d, h2, w2, _ptr(w_in), _ptr(b_in), _ptr(pos), Cw, _ptr(out), _stream()),
           "fv_next_scale_input")
    return out


class FvGenerator:
    """Device copies of `inputs.GenerationTensors` and the fv_generate call for one context."""

    def __init__(self, ctx: "FvContext", gt, tau: float = 1.0):
        dev = ctx.dev
        f32 = lambda a: torch.from_numpy(a).to(dev, torch.float32).contiguous()
        bf = lambda a: torch.from_numpy(a.view("int16")).to(dev).view(torch.bfloat16).contiguous()
        self.ctx = ctx
        self.codebook, self.w_head, self.b_head = f32(gt.codebook), bf(gt.w_head), bf(gt.b_head)
        self.mod_head, self.w_in, self.b_in = f32(gt.mod_head), f32(gt.w_in), f32(gt.b_in)
        self.pos = [f32(p) for p in gt.pos]
        self.V, self.d = self.codebook.shape
        self._pos_arr = (C.c_void_p * len(self.pos))(*[p.data_ptr() for p in self.pos])
        self.gen = fv_generator(self.V, self.d, self.codebook.data_ptr(), self.w_head.data_ptr(), self.b_head.data_ptr(),
                                self.mod_head.data_ptr(), self.w_in.data_ptr(), self.b_in.data_ptr(),
                                C.cast(self._pos_arr, C.POINTER(C.c_void_p)), float(tau))
        nbytes = lib().fv_generate_workspace_bytes(ctx.ctx, C.byref(self.gen))
        self.ws = torch.empty(nbytes + 1024, dtype=torch.uint8, device=dev)
        self.ws_bytes = nbytes

    def generate(self, start: torch.Tensor, keep: Sequence[float], noise: Optional[Sequence[Optional[torch.Tensor]]] = None):
        """start fp32 [B, n_0, C].  Returns (ids per step: list of int32 [B, n_k], r_K fp32 [B, n_K, d])."""
        B = start.shape[0]
        hw = self.ctx.hw
        ns = [h * w for h, w in hw]
        ids = torch.empty(B * sum(ns), dtype=torch.int32, device=start.device)
        r = torch.empty((B, ns[-1], self.d), dtype=torch.float32, device=start.device)
        keep_arr = (C.c_double * len(hw))(*[float(k) for k in keep])
        noise_arr = None
        if noise is not None:
            noise_arr = (C.c_void_p * len(hw))(*[None if t is None else t.data_ptr() for t in noise])
        wsp = (self.ws.data_ptr() + 1023) // 1024 * 1024
        _check(lib().fv_generate(self.ctx.ctx, C.byref(self.gen), _ptr(start), B, keep_arr, noise_arr, _ptr(ids), _ptr(r), wsp,
                                 self.ws_bytes, _stream()), "fv_generate")
        out, off = [], 0
        for n in ns:
            out.append(ids[off:off + B * n].view(B, n))
            off += B * n
        return out, r


class FvContext:
    """Owns the device buffers a context borrows (weights, KV cache, sublayer caches, workspace) and
    forwards to fv_create / fv_var_step / ...  Weights are given as numpy bf16 bit patterns
    (`inputs.ModelTensors`) or as torch bf16 CUDA tensors with the same field names."""

    def __init__(self, L: int, Cw: int, H: int, sides_hw: Sequence[Sequence[int]], cache_step: int, B_max: int,
                 kv_capacity: int, tensors, cross_len: int = 0, mlp_ratio: int = 4, device="cuda:0", granularity: int = 0,
                 rope_base: float = 0.0, interp_mode: int = 0, qk_scale=None, resid_dtype: int = 0):
        self.dev = torch.device(device)
        self.L, self.C, self.H, self.B_max, self.cross_len = L, Cw, H, B_max, cross_len
        self.n_sub = 3 if cross_len else 2
        self.hw = [tuple(s) for s in sides_hw]
        self.kv_capacity = (kv_capacity + 7) // 8 * 8
        self._h = (C.c_int32 * len(self.hw))(*[s[0] for s in self.hw])
        self._w = (C.c_int32 * len(self.hw))(*[s[1] for s in self.hw])
        self.granularity = granularity
        self.cfg = fv_config(L, Cw, H, mlp_ratio, cross_len, B_max, len(self.hw), self._h, self._w, cache_step,
                             self.kv_capacity, granularity, float(rope_base), int(interp_mode), int(resid_dtype))
        self.x_dtype = torch.bfloat16 if resid_dtype == 1 else torch.float32
        self._keep: List[torch.Tensor] = []

        def dev_bf16(a):
            if isinstance(a, torch.Tensor):
                t = a.to(self.dev).contiguous()
            else:
                t = torch.from_numpy(a.view("int16")).to(self.dev).view(torch.bfloat16).contiguous()
            self._keep.append(t)
            return t

        self._arrays = {}
        W = fv_weights()
        for name in ("w_qkv", "b_qkv", "w_o", "b_o", "w_fc1", "b_fc1", "w_fc2", "b_fc2", "w_q_x", "w_kv_x", "w_o_x"):
            lst = getattr(tensors, name)
            if not lst:
                setattr(W, name, None)
                continue
            ts = [dev_bf16(a) for a in lst]
            arr = (C.c_void_p * L)(*[t.data_ptr() for t in ts])
            self._arrays[name] = arr
            setattr(W, name, C.cast(arr, C.POINTER(C.c_void_p)))
        mod = tensors.mod
        self.mod = (mod if isinstance(mod, torch.Tensor) else torch.from_numpy(mod)).to(self.dev, torch.float32).contiguous()
        assert tuple(self.mod.shape) == (L, B_max, 6, Cw)
        W.mod_dev = self.mod.data_ptr()
        self.text = dev_bf16(tensors.text) if cross_len else None
        W.text_dev = self.text.data_ptr() if cross_len else None
        self.qk_scale = None
        if qk_scale is not None:      # [L, H] fp32: cosine attention
            self.qk_scale = (qk_scale if isinstance(qk_scale, torch.Tensor) else torch.from_numpy(qk_scale)).to(self.dev, torch.float32).contiguous()
            assert tuple(self.qk_scale.shape) == (L, H)
        W.qk_scale_dev = self.qk_scale.data_ptr() if self.qk_scale is not None else None
        self.weights = W
        Lb = lib()
        self.kv = torch.empty(Lb.fv_kv_bytes(C.byref(self.cfg)) + 1024, dtype=torch.uint8, device=self.dev)
        self.cache = torch.empty(Lb.fv_cache_bytes(C.byref(self.cfg)) + 1024, dtype=torch.uint8, device=self.dev)
        self.ws = torch.empty(Lb.fv_workspace_bytes(C.byref(self.cfg)) + 1024, dtype=torch.uint8, device=self.dev)
        al = lambda t: (t.data_ptr() + 1023) // 1024 * 1024
        self.ctx = C.c_void_p()
        torch.cuda.synchronize(self.dev)
        _check(Lb.fv_create(C.byref(self.cfg), C.byref(W), al(self.kv), al(self.cache) if cache_step >= 0 else None,
                            al(self.ws), C.byref(self.ctx)), "fv_create")

    def close(self):
        if self.ctx:
            lib().fv_destroy(self.ctx)
            self.ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        _check(lib().fv_reset(self.ctx), "fv_reset")

    def state(self):
        a, b = C.c_int32(), C.c_int32()
        _check(lib().fv_get_state(self.ctx, C.byref(a), C.byref(b)), "fv_get_state")
        return a.value, b.value

    def set_state(self, next_step: int, kv_len: int):
        _check(lib().fv_set_state(self.ctx, next_step, kv_len), "fv_set_state")

    def prepare_text(self, B: int):
        _check(lib().fv_prepare_text(self.ctx, B, _stream()), "fv_prepare_text")

    def device_status(self) -> int:
        """The kernels' status code since the last call (0 = fine); the word is cleared."""
        return self.device_status_pair()[1]

    def device_status_pair(self):
        """(fv_status, code): (0, 0), (FV_ERR_TIMEOUT, 101..105) or (FV_ERR_DEVICE_DATA, 40 / 41)."""
        code = C.c_int32()
        rc = lib().fv_device_status(self.ctx, C.byref(code), _stream())
        if rc not in (0, 6, 7):
            raise FvError(rc, "fv_device_status")
        return rc, code.value

    def selftest_expired_wait(self, limit_ns: int) -> None:
        _check(lib().fv_selftest_expired_wait(self.ctx, int(limit_ns), _stream()), "fv_selftest_expired_wait")

    def kv_views(self, block: int):
        """(K [B_max, cap, C], V^T [B_max, C, cap]) bf16 views of one block's KV cache."""
        kp, vp = C.c_void_p(), C.c_void_p()
        _check(lib().fv_kv_pointers(self.ctx, block, C.byref(kp), C.byref(vp)), "fv_kv_pointers")
        base = self.kv.data_ptr()
        nel = self.B_max * self.kv_capacity * self.C
        kview = self.kv[kp.value - base: kp.value - base + 2 * nel].view(torch.bfloat16).view(self.B_max, self.kv_capacity, self.C)
        vview = self.kv[vp.value - base: vp.value - base + 2 * nel].view(torch.bfloat16).view(self.B_max, self.C, self.kv_capacity)
        return kview, vview

    def cache_view(self, block: int, sublayer: int, B: Optional[int] = None):
        p = C.c_void_p()
        _check(lib().fv_cache_pointer(self.ctx, block, sublayer, C.byref(p)), "fv_cache_pointer")
        hc, wc = self.hw[self.cfg.cache_step]
        B = B or self.B_max
        nel = B * hc * wc * self.C
        off = p.value - self.cache.data_ptr()
        if self.granularity == 1:      # the step-level cache: fp32 output map of the caching step
            return self.cache[off: off + 4 * nel].view(torch.float32).view(B, hc * wc, self.C)
        return self.cache[off: off + 2 * nel].view(torch.bfloat16).view(B, hc * wc, self.C)

    def var_step_host(self, tokens_host: torch.Tensor, scale_idx: int, keep_ratio: float, out_host: torch.Tensor) -> torch.Tensor:
        """fv_var_step_host: token maps in (pinned) host memory; the step runs on the current stream, the copies on the
        context's own streams.  Call host_io_flush() and synchronise before reading out_host."""
        assert not tokens_host.is_cuda and not out_host.is_cuda and tokens_host.dtype == self.x_dtype and out_host.dtype == self.x_dtype
        assert tokens_host.is_contiguous() and out_host.is_contiguous()
        if getattr(self, "_staging", None) is None:
            nbytes = lib().fv_var_step_host_staging_bytes(C.byref(self.cfg))
            self._staging = torch.empty(nbytes + 1024, dtype=torch.uint8, device=self.dev)
            self._staging_bytes = nbytes
        sp = (self._staging.data_ptr() + 1023) // 1024 * 1024
        _check(lib().fv_var_step_host(self.ctx, tokens_host.data_ptr(), tokens_host.shape[0], scale_idx, float(keep_ratio),
                                      out_host.data_ptr(), sp, self._staging_bytes, _stream()), "fv_var_step_host")
        return out_host

    def host_io_flush(self) -> None:
        _check(lib().fv_host_io_flush(self.ctx, _stream()), "fv_host_io_flush")

    def var_step(self, tokens: torch.Tensor, scale_idx: int, keep_ratio: float, out: Optional[torch.Tensor] = None,
                 forced_idx: Optional[torch.Tensor] = None, idx_trace: Optional[torch.Tensor] = None) -> torch.Tensor:
        assert tokens.dtype == self.x_dtype, "token maps take the context's residual-stream type"
        B = tokens.shape[0]
        if out is None:
            out = torch.empty_like(tokens)
        _check(lib().fv_var_step(self.ctx, _ptr(tokens), B, scale_idx, float(keep_ratio), _ptr(out), _ptr(forced_idx),
                                 _ptr(idx_trace), _stream()), "fv_var_step")
        return out
