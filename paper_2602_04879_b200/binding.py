"""ctypes binding of libdppo.so: argument marshalling only.

Every function mirrors the C entry point of the same name in include/dppo.h and takes torch
tensors for the pointer arguments (CUDA tensors for the device entry points, CPU tensors for the
``_host`` one).  Nothing is computed here; if the library is missing or cannot be loaded the
import of a symbol raises, there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, c_char_p, c_float, c_int, c_int32, c_int64, c_size_t, c_void_p

import torch

BINARY_TV, BINARY_KL, TOPK_TV, TOPK_KL, PPO_CLIP, MINIMAL_MASK, GIVEN_D = 0, 1, 2, 3, 4, 5, 6
F32, BF16 = 0, 1
DLOGITS_SAME, DLOGITS_F32 = 0, 1
KERNEL_AUTO, KERNEL_GENERIC, KERNEL_RING = 0, 1, 2
INJECT_NO_COPIES = 1
STATUS_BAD_SAMPLED_ID, STATUS_BAD_TOPK_ID, STATUS_NONFINITE_ROW, STATUS_WAIT_LIMIT = 1, 2, 4, 8
VARIANTS = {"binary_tv": BINARY_TV, "binary_kl": BINARY_KL, "topk_tv": TOPK_TV, "topk_kl": TOPK_KL, "ppo_clip": PPO_CLIP, "minimal_mask": MINIMAL_MASK, "given_d": GIVEN_D}

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libdppo.so")
_lib = None


class DppoOpts(ctypes.Structure):
    """dppo_opts of include/dppo.h (all-zero = defaults)."""
    _fields_ = [("loss_scale", c_float), ("dlogits_dtype", c_int), ("kernel", c_int), ("is_cap", c_float), ("eps_low", c_float),
                ("lm_head_layout", c_int), ("gemm_cta_group", c_int), ("fused_rows_per_block", c_int), ("wait_limit_us", c_int),
                ("test_inject", c_int), ("fused_two_pass", c_int), ("row_cluster", c_int)]


def _opts(loss_scale=0.0, dlogits_f32=False, kernel=KERNEL_AUTO, is_cap=0.0, eps_low=0.0, w_is_vd=False, cta_group=0,
          rows_per_block=0, wait_limit_us=0, test_inject=0, two_pass=False, row_cluster=0):
    return DppoOpts(float(loss_scale), DLOGITS_F32 if dlogits_f32 else DLOGITS_SAME, int(kernel), float(is_cap), float(eps_low),
                    1 if w_is_vd else 0, int(cta_group), int(rows_per_block), int(wait_limit_us), int(test_inject),
                    1 if two_pass else 0, int(row_cluster))


class DppoError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {error_string(code)} ({code})")


def lib():
    """The loaded library (loads it on first use; raises if it is not built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2602_04879_b200.build` (there is no fallback path)")
        L = ctypes.CDLL(_LIB_PATH)
        L.dppo_version.restype = c_int
        L.dppo_opts_size.restype = c_size_t
        if int(L.dppo_opts_size()) != ctypes.sizeof(DppoOpts):
            raise RuntimeError(f"{_LIB_PATH}: dppo_opts is {int(L.dppo_opts_size())} bytes in the library, {ctypes.sizeof(DppoOpts)} in this binding "
                               "(rebuild the library: `python -m paper_2602_04879_b200.build`)")
        L.dppo_error_string.restype = c_char_p
        L.dppo_error_string.argtypes = [c_int]
        L.dppo_workspace_bytes.restype = c_size_t
        L.dppo_workspace_bytes.argtypes = [c_int64, c_int64, c_int, c_int]
        L.dppo_loss_fwd_bwd.restype = c_int
        L.dppo_loss_fwd_bwd.argtypes = [c_void_p, c_int64, c_int64, c_int64, c_int, c_void_p, c_void_p, c_void_p, c_void_p,
                                        c_void_p, c_void_p, c_int, c_int, c_float, POINTER(DppoOpts),
                                        c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_void_p, c_void_p,
                                        c_void_p, c_size_t, c_void_p]
        L.dppo_host_staging_bytes.restype = c_size_t
        L.dppo_host_staging_bytes.argtypes = [c_int64, c_int64, c_int, c_int, c_int]
        L.dppo_loss_fwd_bwd_host.restype = c_int
        L.dppo_loss_fwd_bwd_host.argtypes = [c_void_p, c_int64, c_int64, c_int, c_void_p, c_void_p, c_void_p, c_void_p,
                                             c_void_p, c_void_p, c_int, c_int, c_float, POINTER(DppoOpts),
                                             c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                             c_void_p, c_size_t, c_int64]
        L.dppo_fused_workspace_bytes.restype = c_size_t
        L.dppo_fused_workspace_bytes.argtypes = [c_int64, c_int64, c_int64, c_int]
        L.dppo_fused_lmhead_fwd_bwd.restype = c_int
        L.dppo_fused_lmhead_fwd_bwd.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_void_p, c_void_p, c_void_p,
                                                c_void_p, c_void_p, c_void_p, c_int, c_int, c_float, POINTER(DppoOpts),
                                                c_void_p, c_void_p, c_void_p,
                                                c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
        L.dppo_exact_divergence.restype = c_int
        L.dppo_exact_divergence.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int64, c_int, c_void_p, c_void_p,
                                            c_void_p, c_void_p, c_void_p, POINTER(DppoOpts), c_void_p]
        L.dppo_gemm_tn_bf16.restype = c_int
        L.dppo_gemm_tn_bf16.argtypes = [c_void_p, c_int64, c_void_p, c_int64, c_int, c_int, c_int, c_void_p, c_int64,
                                        c_void_p, POINTER(DppoOpts), c_void_p]
        L.dppo_gemm_nn_bf16.restype = c_int
        L.dppo_gemm_nn_bf16.argtypes = L.dppo_gemm_tn_bf16.argtypes
        L.dppo_loss_fwd_bwd_static_ws.restype = c_int
        L.dppo_loss_fwd_bwd_static_ws.argtypes = L.dppo_loss_fwd_bwd.argtypes[:22] + [c_void_p]
        _lib = L
    return _lib


def version():
    return int(lib().dppo_version())


def error_string(code):
    return lib().dppo_error_string(int(code)).decode()


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _dtype_code(t):
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"logits dtype {t.dtype} not supported (float32 or bfloat16)")


def dppo_workspace_bytes(T, V=1, K=0, variant=BINARY_TV):
    return int(lib().dppo_workspace_bytes(int(T), int(V), int(K), int(variant)))


def _divergence_buffer(T, dev, variant, given):
    """The call's divergence buffer: an output, and for GIVEN_D also the input (a copy of the caller's values)."""
    if int(variant) == GIVEN_D:
        assert given is not None and given.is_cuda and given.dtype == torch.float32 and given.shape == (T,), "given_divergence"
        return given.contiguous().clone()
    return torch.empty(T, dtype=torch.float32, device=dev)


def dppo_loss_fwd_bwd(logits, sampled_ids, mu_logp, advantages, token_mask=None, variant=BINARY_TV, K=0, delta=0.2,
                      mu_topk_ids=None, mu_topk_p=None, loss_scale=0.0, dlogits_f32=False, kernel=KERNEL_AUTO,
                      dlogits=None, want_stats=False, workspace=None, status=None, stream=None, is_cap=0.0, eps_low=0.0,
                      given_divergence=None, wait_limit_us=0, test_inject=0, row_cluster=0):
    """Calls ``dppo_loss_fwd_bwd`` on CUDA tensors.  Output tensors are allocated with torch unless
    given.  Returns dict(loss[1], divergence[T], mask[T], dlogits[T,V], stats[8] or None, status[1]);
    nothing is synchronised.  ``given_divergence`` [T] fp32: the per-token divergence for variant GIVEN_D (copied into
    the in/out divergence buffer of the call)."""
    assert logits.is_cuda and logits.dim() == 2 and logits.stride(1) == 1
    T, V = logits.shape
    dev = logits.device
    out_dtype = torch.float32 if dlogits_f32 else logits.dtype
    if dlogits is None:
        dlogits = torch.empty((T, V), dtype=out_dtype, device=dev)
    assert dlogits.dtype == out_dtype and dlogits.stride(1) == 1
    loss = torch.empty(1, dtype=torch.float32, device=dev)
    D = _divergence_buffer(T, dev, variant, given_divergence)
    M = torch.empty(T, dtype=torch.uint8, device=dev)
    stats = torch.empty(8, dtype=torch.float32, device=dev) if want_stats else None
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    nbytes = dppo_workspace_bytes(T, V, K, variant)
    if workspace is None:
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    for name, t, dt in (("sampled_ids", sampled_ids, torch.int32), ("mu_logp", mu_logp, torch.float32),
                        ("advantages", advantages, torch.float32), ("token_mask", token_mask, torch.uint8),
                        ("mu_topk_ids", mu_topk_ids, torch.int32), ("mu_topk_p", mu_topk_p, torch.float32)):
        if t is not None:
            assert t.is_cuda and t.dtype == dt and t.is_contiguous(), name
    opts = _opts(loss_scale, dlogits_f32, kernel, is_cap, eps_low, wait_limit_us=wait_limit_us, test_inject=test_inject,
                 row_cluster=row_cluster)
    st = stream if stream is not None else torch.cuda.current_stream(dev)
    with torch.cuda.device(dev):
        rc = lib().dppo_loss_fwd_bwd(_ptr(logits), T, V, logits.stride(0) if T > 0 else V, _dtype_code(logits),
                                     _ptr(sampled_ids), _ptr(mu_logp), _ptr(mu_topk_ids), _ptr(mu_topk_p),
                                     _ptr(advantages), _ptr(token_mask), int(variant), int(K), float(delta),
                                     ctypes.byref(opts), _ptr(loss), _ptr(D), _ptr(M), _ptr(dlogits),
                                     dlogits.stride(0) if T > 0 else V, _ptr(stats), _ptr(status), _ptr(workspace),
                                     workspace.numel(), c_void_p(st.cuda_stream))
    if rc != 0:
        raise DppoError(rc, "dppo_loss_fwd_bwd")
    return dict(loss=loss, divergence=D, mask=M, dlogits=dlogits, stats=stats, status=status)


def dppo_fused_workspace_bytes(T, d, V, K=0):
    return int(lib().dppo_fused_workspace_bytes(int(T), int(d), int(V), int(K)))


def dppo_fused_lmhead_fwd_bwd(hidden, W, sampled_ids, mu_logp, advantages, token_mask=None, variant=BINARY_TV, delta=0.2,
                              loss_scale=0.0, want_stats=False, workspace=None, dHidden=None, dW=None, status=None, stream=None,
                              is_cap=0.0, eps_low=0.0, K=0, mu_topk_ids=None, mu_topk_p=None, given_divergence=None, w_is_vd=False,
                              cta_group=0, rows_per_block=0, wait_limit_us=0, test_inject=0, two_pass=False):
    """Calls ``dppo_fused_lmhead_fwd_bwd`` on CUDA tensors: hidden [T,d] bf16, W [d,V] bf16.  Returns
    dict(loss[1], divergence[T], mask[T], dHidden[T,d] fp32, dW[d,V] fp32, stats, status); nothing is synchronised.
    ``given_divergence``: as for ``dppo_loss_fwd_bwd`` (variant GIVEN_D).  ``w_is_vd``: W (and dW) are [V,d], the layout
    of a linear layer's weight, instead of [d,V].  ``cta_group``, ``rows_per_block``, ``wait_limit_us``, ``test_inject``: the
    fields of dppo_opts of the same names (``rows_per_block`` = fused_rows_per_block, ``two_pass`` = fused_two_pass)."""
    assert hidden.is_cuda and W.is_cuda and hidden.dtype == torch.bfloat16 and W.dtype == torch.bfloat16
    assert hidden.is_contiguous() and W.is_contiguous() and hidden.shape[1] == W.shape[1 if w_is_vd else 0]
    T, d = hidden.shape
    V = W.shape[0 if w_is_vd else 1]
    dev = hidden.device
    loss = torch.empty(1, dtype=torch.float32, device=dev)
    D = _divergence_buffer(T, dev, variant, given_divergence)
    M = torch.empty(T, dtype=torch.uint8, device=dev)
    if dHidden is None:
        dHidden = torch.empty((T, d), dtype=torch.float32, device=dev)
    if dW is None:
        dW = torch.empty((V, d) if w_is_vd else (d, V), dtype=torch.float32, device=dev)
    stats = torch.empty(8, dtype=torch.float32, device=dev) if want_stats else None
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    if workspace is None:
        rows = min(T, rows_per_block) if rows_per_block > 0 else T
        workspace = torch.empty(dppo_fused_workspace_bytes(rows, d, V, K), dtype=torch.uint8, device=dev)
    opts = _opts(loss_scale, False, 0, is_cap, eps_low, w_is_vd, cta_group, rows_per_block, wait_limit_us, test_inject, two_pass)
    st = stream if stream is not None else torch.cuda.current_stream(dev)
    with torch.cuda.device(dev):
        rc = lib().dppo_fused_lmhead_fwd_bwd(_ptr(hidden), _ptr(W), T, d, V, _ptr(sampled_ids), _ptr(mu_logp),
                                             _ptr(mu_topk_ids), _ptr(mu_topk_p), _ptr(advantages),
                                             _ptr(token_mask), int(variant), int(K), float(delta), ctypes.byref(opts), _ptr(loss),
                                             _ptr(D), _ptr(M), _ptr(dHidden), _ptr(dW), _ptr(stats), _ptr(status),
                                             _ptr(workspace), workspace.numel(), c_void_p(st.cuda_stream))
    if rc != 0:
        raise DppoError(rc, "dppo_fused_lmhead_fwd_bwd")
    return dict(loss=loss, divergence=D, mask=M, dHidden=dHidden, dW=dW, stats=stats, status=status)


def dppo_exact_divergence(logits, mu_logits, token_mask=None, status=None, stream=None, want_tv=True, wait_limit_us=0,
                          test_inject=0):
    """Calls ``dppo_exact_divergence``: per-row exact TV, KL(mu||pi) and entropy of pi from two [T,V] CUDA logits tensors
    of the same dtype.  Returns dict(tv, kl, entropy, status); ``want_tv=False`` passes tv = NULL (one sweep, tv is None)."""
    assert logits.is_cuda and mu_logits.is_cuda and logits.dtype == mu_logits.dtype and logits.shape == mu_logits.shape
    assert logits.stride(1) == 1 and mu_logits.stride(1) == 1
    T, V = logits.shape
    dev = logits.device
    tv = torch.empty(T, dtype=torch.float32, device=dev) if want_tv else None
    kl = torch.empty(T, dtype=torch.float32, device=dev)
    ent = torch.empty(T, dtype=torch.float32, device=dev)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    st = stream if stream is not None else torch.cuda.current_stream(dev)
    opts = _opts(wait_limit_us=wait_limit_us, test_inject=test_inject)
    with torch.cuda.device(dev):
        rc = lib().dppo_exact_divergence(_ptr(logits), _ptr(mu_logits), T, V, logits.stride(0) if T > 0 else V,
                                         mu_logits.stride(0) if T > 0 else V, _dtype_code(logits), _ptr(token_mask), _ptr(tv),
                                         _ptr(kl), _ptr(ent), _ptr(status), ctypes.byref(opts), c_void_p(st.cuda_stream))
    if rc != 0:
        raise DppoError(rc, "dppo_exact_divergence")
    return dict(tv=tv, kl=kl, entropy=ent, status=status)


def dppo_gemm_tn_bf16(A, B, C=None, status=None, stream=None, cta_group=0, wait_limit_us=0, test_inject=0):
    """C[M,N] fp32 = A[M,K] . B[N,K]^T for bf16 CUDA matrices (last dimension contiguous)."""
    assert A.is_cuda and B.is_cuda and A.dtype == torch.bfloat16 and B.dtype == torch.bfloat16
    assert A.stride(1) == 1 and B.stride(1) == 1 and A.shape[1] == B.shape[1]
    M, K = A.shape
    N = B.shape[0]
    if C is None:
        C = torch.empty((M, N), dtype=torch.float32, device=A.device)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=A.device)
    st = stream if stream is not None else torch.cuda.current_stream(A.device)
    with torch.cuda.device(A.device):
        rc = lib().dppo_gemm_tn_bf16(_ptr(A), A.stride(0), _ptr(B), B.stride(0), M, N, K, _ptr(C), C.stride(0), _ptr(status),
                                     ctypes.byref(_opts(cta_group=cta_group, wait_limit_us=wait_limit_us, test_inject=test_inject)),
                                     c_void_p(st.cuda_stream))
    if rc != 0:
        raise DppoError(rc, "dppo_gemm_tn_bf16")
    return C, status


def dppo_gemm_nn_bf16(A, B, C=None, status=None, stream=None, cta_group=0, wait_limit_us=0, test_inject=0):
    """C[M,N] fp32 = A[M,K] . B[K,N] for bf16 CUDA matrices (last dimension contiguous)."""
    assert A.is_cuda and B.is_cuda and A.dtype == torch.bfloat16 and B.dtype == torch.bfloat16
    assert A.stride(1) == 1 and B.stride(1) == 1 and A.shape[1] == B.shape[0]
    M, K = A.shape
    N = B.shape[1]
    if C is None:
        C = torch.empty((M, N), dtype=torch.float32, device=A.device)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=A.device)
    st = stream if stream is not None else torch.cuda.current_stream(A.device)
    with torch.cuda.device(A.device):
        rc = lib().dppo_gemm_nn_bf16(_ptr(A), A.stride(0), _ptr(B), B.stride(0), M, N, K, _ptr(C), C.stride(0), _ptr(status),
                                     ctypes.byref(_opts(cta_group=cta_group, wait_limit_us=wait_limit_us, test_inject=test_inject)),
                                     c_void_p(st.cuda_stream))
    if rc != 0:
        raise DppoError(rc, "dppo_gemm_nn_bf16")
    return C, status


STATIC_WS_MAX_ROWS = 65536


def dppo_loss_fwd_bwd_static_ws(logits, sampled_ids, mu_logp, advantages, token_mask=None, variant=BINARY_TV, K=0,
                                delta=0.2, mu_topk_ids=None, mu_topk_p=None, loss_scale=0.0, dlogits_f32=False,
                                kernel=KERNEL_AUTO, out=None, stream=None, is_cap=0.0, eps_low=0.0, given_divergence=None):
    """Calls ``dppo_loss_fwd_bwd_static_ws``: the same operation with the scratch taken from the array
    built into the library, for callers that cannot allocate device memory.  This wrapper does not
    allocate either when ``out`` holds the output tensors (loss[1], divergence[T], mask[T],
    dlogits[T,V], status[1], optionally stats[8]); without ``out`` it creates them with torch for
    convenience.  At most ``STATIC_WS_MAX_ROWS`` rows per call; calls that may overlap on the GPU race on
    the shared array.  ``given_divergence`` (variant GIVEN_D): without ``out`` it is copied into the new
    divergence buffer; with ``out`` the caller fills ``out["divergence"]`` itself."""
    assert logits.is_cuda and logits.dim() == 2 and logits.stride(1) == 1
    T, V = logits.shape
    dev = logits.device
    if out is None:
        out = dict(loss=torch.empty(1, dtype=torch.float32, device=dev),
                   divergence=_divergence_buffer(T, dev, variant, given_divergence),
                   mask=torch.empty(T, dtype=torch.uint8, device=dev),
                   dlogits=torch.empty((T, V), dtype=torch.float32 if dlogits_f32 else logits.dtype, device=dev),
                   status=torch.zeros(1, dtype=torch.int32, device=dev), stats=None)
    dl = out["dlogits"]
    opts = _opts(loss_scale, dlogits_f32, kernel, is_cap, eps_low)
    st = stream if stream is not None else torch.cuda.current_stream(dev)
    with torch.cuda.device(dev):
        rc = lib().dppo_loss_fwd_bwd_static_ws(_ptr(logits), T, V, logits.stride(0) if T > 0 else V, _dtype_code(logits),
                                               _ptr(sampled_ids), _ptr(mu_logp), _ptr(mu_topk_ids), _ptr(mu_topk_p),
                                               _ptr(advantages), _ptr(token_mask), int(variant), int(K), float(delta),
                                               ctypes.byref(opts), _ptr(out["loss"]), _ptr(out["divergence"]),
                                               _ptr(out["mask"]), _ptr(dl), dl.stride(0) if T > 0 else V,
                                               _ptr(out.get("stats")), _ptr(out["status"]), c_void_p(st.cuda_stream))
    if rc != 0:
        raise DppoError(rc, "dppo_loss_fwd_bwd_static_ws")
    return out


def dppo_host_staging_bytes(rows_per_chunk, V, K, logits_dtype, dlogits_f32=False):
    return int(lib().dppo_host_staging_bytes(int(rows_per_chunk), int(V), int(K), int(logits_dtype),
                                             DLOGITS_F32 if dlogits_f32 else DLOGITS_SAME))


def dppo_loss_fwd_bwd_host(logits, sampled_ids, mu_logp, advantages, token_mask=None, variant=BINARY_TV, K=0, delta=0.2,
                           mu_topk_ids=None, mu_topk_p=None, loss_scale=0.0, dlogits_f32=False, kernel=KERNEL_AUTO,
                           rows_per_chunk=1024, staging=None, want_dlogits=False, device="cuda:0", out=None, is_cap=0.0, eps_low=0.0):
    """Calls ``dppo_loss_fwd_bwd_host`` on CPU tensors (pinned recommended); ``staging`` is a CUDA
    uint8 tensor of at least ``dppo_host_staging_bytes`` bytes (allocated here if None).  Returns
    dict(loss(float), divergence, mask, dlogits or None, status(int)) with host tensors."""
    assert not logits.is_cuda and logits.dim() == 2 and logits.is_contiguous()
    T, V = logits.shape
    dt = _dtype_code(logits)
    need = dppo_host_staging_bytes(rows_per_chunk, V, K if variant in (TOPK_TV, TOPK_KL) else 0, dt, dlogits_f32)
    if staging is None:
        staging = torch.empty(need, dtype=torch.uint8, device=device)
    out = out or {}
    D = out.get("divergence")
    if D is None:
        D = torch.empty(T, dtype=torch.float32).pin_memory()
    M = out.get("mask")
    if M is None:
        M = torch.empty(T, dtype=torch.uint8).pin_memory()
    dl = None
    if want_dlogits:
        dl = out.get("dlogits")
        if dl is None:
            dl = torch.empty((T, V), dtype=torch.float32 if dlogits_f32 else logits.dtype).pin_memory()
    loss = c_float(0.0)
    status = c_int32(0)
    opts = _opts(loss_scale, dlogits_f32, kernel, is_cap, eps_low)
    with torch.cuda.device(staging.device):
        rc = lib().dppo_loss_fwd_bwd_host(_ptr(logits), T, V, dt, _ptr(sampled_ids), _ptr(mu_logp), _ptr(mu_topk_ids),
                                          _ptr(mu_topk_p), _ptr(advantages), _ptr(token_mask), int(variant), int(K),
                                          float(delta), ctypes.byref(opts), ctypes.byref(loss), _ptr(D), _ptr(M),
                                          _ptr(dl), ctypes.byref(status), _ptr(staging), staging.numel(),
                                          int(rows_per_chunk))
    if rc != 0:
        raise DppoError(rc, "dppo_loss_fwd_bwd_host")
    return dict(loss=float(loss.value), divergence=D, mask=M, dlogits=dl, status=int(status.value))
