"""Python binding of the NAT C-ABI library (ctypes; argument marshalling only).

Every function here has the name and the meaning of the C entry point it
calls (see include/nat.h).  torch tensors supply device memory and the current
CUDA stream; all arithmetic runs in the library's kernels.  There is no CPU
fallback: loading fails loudly when the shared library is missing.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libnat_b200.so")

NAT_SEL_URS, NAT_SEL_RPC, NAT_SEL_DET = 0, 1, 2
NAT_F32, NAT_BF16 = 0, 1
NAT_DEV_TIMEOUT, NAT_DEV_CAPACITY, NAT_DEV_FALLBACK, NAT_DEV_BAD_TARGET = 1, 2, 4, 8

SYMBOLS = (
    "nat_status_string", "nat_last_error", "nat_version", "nat_grpo_adv", "nat_select",
    "nat_compact_workspace_bytes", "nat_compact", "nat_policy_loss_workspace_bytes",
    "nat_policy_loss_fwd", "nat_policy_loss_bwd", "nat_compact_static",
    "nat_compact_static_max_tokens", "nat_policy_loss_fwd_bwd", "nat_trace_begin",
    "nat_trace_end", "nat_select_survival", "nat_gather_rows", "nat_scatter_rows",
    "nat_poll_status", "nat_compact_prefix", "nat_select_cutlaw",
    "nat_select_cutlaw_workspace_bytes",
)
TRACE_KINDS = ("fwd", "dz", "dh", "dw", "e")


class NatError(RuntimeError):
    pass


class SelectParams(ctypes.Structure):
    _fields_ = [("mode", ctypes.c_int32), ("min_cut", ctypes.c_int32), ("p", ctypes.c_double),
                ("beta", ctypes.c_double), ("seed", ctypes.c_uint64), ("offset", ctypes.c_uint64),
                ("resp_base", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class LossParams(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("V", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("B", ctypes.c_int32), ("clip_lo", ctypes.c_float), ("clip_hi", ctypes.c_float),
                ("hidden_is_compact", ctypes.c_int32), ("accumulate_dW", ctypes.c_int32),
                ("kl_beta", ctypes.c_float), ("reserved", ctypes.c_int32),
                ("ref_logp", ctypes.c_void_p)]


_lib = None


def load():
    """dlopen the library (built in-tree by ``build.build()``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise NatError(f"{LIB_PATH} is missing: run `python -m paper_2603_06619_b200.build` "
                       "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
    lib.nat_status_string.restype = ctypes.c_char_p
    lib.nat_status_string.argtypes = [ctypes.c_int]
    lib.nat_last_error.restype = ctypes.c_char_p
    lib.nat_version.restype = ctypes.c_int
    lib.nat_grpo_adv.argtypes = [i32, i32, vp, f32, vp, vp]
    lib.nat_select.argtypes = [ctypes.POINTER(SelectParams), i32, vp, i64, vp, vp, vp, vp]
    lib.nat_select_survival.argtypes = [i32, vp, i64, vp, ctypes.c_uint64, ctypes.c_uint64, i32,
                                        vp, vp, vp]
    lib.nat_select_survival.restype = ctypes.c_int
    lib.nat_select_cutlaw_workspace_bytes.restype = ctypes.c_size_t
    lib.nat_select_cutlaw_workspace_bytes.argtypes = [i32, i64]
    lib.nat_select_cutlaw.argtypes = [i32, vp, i64, vp, ctypes.c_uint64, ctypes.c_uint64, i32, vp,
                                      vp, vp, vp, ctypes.c_size_t, vp]
    lib.nat_select_cutlaw.restype = ctypes.c_int
    lib.nat_compact_prefix.argtypes = [i32, vp, i64, vp, vp, vp, vp, vp, i64, vp]
    lib.nat_compact_prefix.restype = ctypes.c_int
    lib.nat_poll_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.nat_poll_status.restype = ctypes.c_int
    lib.nat_gather_rows.argtypes = [vp, i64, vp, vp, i64, vp, vp]
    lib.nat_gather_rows.restype = ctypes.c_int
    lib.nat_scatter_rows.argtypes = [vp, i64, vp, vp, i64, i64, vp, vp]
    lib.nat_scatter_rows.restype = ctypes.c_int
    lib.nat_compact_workspace_bytes.restype = ctypes.c_size_t
    lib.nat_compact_workspace_bytes.argtypes = [i64]
    lib.nat_compact.argtypes = [i32, vp, i64, vp, vp, vp, vp, vp, i64, vp, ctypes.c_size_t, vp]
    lib.nat_compact_static_max_tokens.restype = ctypes.c_int64
    lib.nat_compact_static.argtypes = [i32, vp, i64, vp, vp, vp, vp, vp, i64, vp]
    lib.nat_compact_static.restype = ctypes.c_int
    lib.nat_policy_loss_workspace_bytes.restype = ctypes.c_size_t
    lib.nat_policy_loss_workspace_bytes.argtypes = [ctypes.POINTER(LossParams), i64]
    lib.nat_policy_loss_fwd.argtypes = [ctypes.POINTER(LossParams)] + [vp] * 10 + [i64] + \
        [vp] * 4 + [ctypes.c_size_t, vp]
    lib.nat_policy_loss_bwd.argtypes = [ctypes.POINTER(LossParams)] + [vp] * 10 + [i64] + \
        [vp] * 6 + [ctypes.c_size_t, vp]
    lib.nat_policy_loss_fwd_bwd.argtypes = [ctypes.POINTER(LossParams)] + [vp] * 10 + [i64] + \
        [vp] * 7 + [ctypes.c_size_t, vp]
    lib.nat_trace_begin.restype = ctypes.c_int
    lib.nat_trace_end.restype = ctypes.c_int
    lib.nat_trace_end.argtypes = [vp, vp]
    for name in ("nat_grpo_adv", "nat_select", "nat_compact", "nat_policy_loss_fwd",
                 "nat_policy_loss_bwd", "nat_policy_loss_fwd_bwd"):
        getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def _check(status):
    if status != 0:
        lib = load()
        raise NatError(f"{lib.nat_status_string(status).decode()}: {lib.nat_last_error().decode()}")


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_contiguous(), "tensors passed to the library must be contiguous"
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def nat_grpo_adv(P, G, rewards, eps, adv):
    _check(load().nat_grpo_adv(P, G, _ptr(rewards), eps, _ptr(adv), _stream()))


def select_params(mode, p=1.0, min_cut=1, beta=1.0, seed=0, offset=0, resp_base=0):
    mode = {"urs": NAT_SEL_URS, "rpc": NAT_SEL_RPC, "det": NAT_SEL_DET}.get(mode, mode)
    return SelectParams(mode=mode, min_cut=min_cut, p=p, beta=beta, seed=seed, offset=offset,
                        resp_base=resp_base, reserved=0)


def nat_select(params, B, cu_seqlens, n_tot, mask, pi, cut_len):
    _check(load().nat_select(ctypes.byref(params), B, _ptr(cu_seqlens), n_tot, _ptr(mask),
                             _ptr(pi), _ptr(cut_len), _stream()))


def nat_select_survival(B, cu_seqlens, n_tot, surv, seed, offset, mask, cut_len, resp_base=0):
    _check(load().nat_select_survival(B, _ptr(cu_seqlens), n_tot, _ptr(surv), seed, offset,
                                      resp_base, _ptr(mask), _ptr(cut_len), _stream()))


def nat_select_cutlaw_workspace_bytes(B, n_tot):
    return load().nat_select_cutlaw_workspace_bytes(B, n_tot)


def nat_select_cutlaw(B, cu_seqlens, n_tot, q, seed, offset, mask, pi, cut_len, workspace,
                      resp_base=0):
    _check(load().nat_select_cutlaw(B, _ptr(cu_seqlens), n_tot, _ptr(q), seed, offset, resp_base,
                                    _ptr(mask), _ptr(pi), _ptr(cut_len), _ptr(workspace),
                                    workspace.numel() * workspace.element_size(), _stream()))


def _row_bytes(t):
    return t.stride(0) * t.element_size() if t.dim() > 1 else t.element_size()


def nat_gather_rows(src, sel_idx, n_sel, cap, dst):
    _check(load().nat_gather_rows(_ptr(src), _row_bytes(src), _ptr(sel_idx), _ptr(n_sel), cap,
                                  _ptr(dst), _stream()))


def nat_scatter_rows(src, sel_idx, n_sel, cap, n_tot, dst):
    _check(load().nat_scatter_rows(_ptr(src), _row_bytes(src), _ptr(sel_idx), _ptr(n_sel), cap,
                                   n_tot, _ptr(dst), _stream()))


def nat_compact_workspace_bytes(n_tot):
    return load().nat_compact_workspace_bytes(n_tot)


def nat_compact(B, cu_seqlens, n_tot, mask, sel_idx, sel_resp, sel_offsets, n_sel, cap, workspace):
    _check(load().nat_compact(B, _ptr(cu_seqlens), n_tot, _ptr(mask), _ptr(sel_idx),
                              _ptr(sel_resp), _ptr(sel_offsets), _ptr(n_sel), cap,
                              _ptr(workspace), workspace.numel() * workspace.element_size(),
                              _stream()))


def nat_compact_prefix(B, cu_seqlens, n_tot, cut_len, sel_idx, sel_resp, sel_offsets, n_sel, cap):
    _check(load().nat_compact_prefix(B, _ptr(cu_seqlens), n_tot, _ptr(cut_len), _ptr(sel_idx),
                                     _ptr(sel_resp), _ptr(sel_offsets), _ptr(n_sel), cap,
                                     _stream()))


def nat_compact_static_max_tokens():
    return load().nat_compact_static_max_tokens()


def nat_compact_static(B, cu_seqlens, n_tot, mask, sel_idx, sel_resp, sel_offsets, n_sel, cap):
    """nat_compact for callers that may not allocate: the scratch is a fixed array
    inside the library (shared by all calls on the GPU, so do not overlap calls)."""
    _check(load().nat_compact_static(B, _ptr(cu_seqlens), n_tot, _ptr(mask), _ptr(sel_idx),
                                     _ptr(sel_resp), _ptr(sel_offsets), _ptr(n_sel), cap,
                                     _stream()))


def loss_params(d, V, dtype, B, clip_lo=0.2, clip_hi=0.2, hidden_is_compact=False,
                accumulate_dW=False, kl_beta=0.0, ref_logp=None):
    """ref_logp (float32 device tensor [n_tot]) must outlive the calls that use the params."""
    dtype = {torch.float32: NAT_F32, torch.bfloat16: NAT_BF16}.get(dtype, dtype)
    return LossParams(d=d, V=V, dtype=dtype, B=B, clip_lo=clip_lo, clip_hi=clip_hi,
                      hidden_is_compact=int(hidden_is_compact), accumulate_dW=int(accumulate_dW),
                      kl_beta=kl_beta, reserved=0, ref_logp=_ptr(ref_logp))


def nat_policy_loss_workspace_bytes(params, n_sel_cap):
    return load().nat_policy_loss_workspace_bytes(ctypes.byref(params), n_sel_cap)


def nat_policy_loss_fwd(params, hidden, W, targets, old_logp, adv, pi, cu_seqlens, sel_idx,
                        sel_resp, n_sel, n_sel_cap, loss, logp, lse, workspace):
    _check(load().nat_policy_loss_fwd(
        ctypes.byref(params), _ptr(hidden), _ptr(W), _ptr(targets), _ptr(old_logp), _ptr(adv),
        _ptr(pi), _ptr(cu_seqlens), _ptr(sel_idx), _ptr(sel_resp), _ptr(n_sel), n_sel_cap,
        _ptr(loss), _ptr(logp), _ptr(lse), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _stream()))


def nat_policy_loss_bwd(params, hidden, W, targets, old_logp, adv, pi, cu_seqlens, sel_idx,
                        sel_resp, n_sel, n_sel_cap, logp, lse, dloss, dHidden, dW, workspace):
    _check(load().nat_policy_loss_bwd(
        ctypes.byref(params), _ptr(hidden), _ptr(W), _ptr(targets), _ptr(old_logp), _ptr(adv),
        _ptr(pi), _ptr(cu_seqlens), _ptr(sel_idx), _ptr(sel_resp), _ptr(n_sel), n_sel_cap,
        _ptr(logp), _ptr(lse), _ptr(dloss), _ptr(dHidden), _ptr(dW), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _stream()))


def nat_policy_loss_fwd_bwd(params, hidden, W, targets, old_logp, adv, pi, cu_seqlens, sel_idx,
                            sel_resp, n_sel, n_sel_cap, dloss, loss, logp, lse, dHidden, dW,
                            workspace):
    _check(load().nat_policy_loss_fwd_bwd(
        ctypes.byref(params), _ptr(hidden), _ptr(W), _ptr(targets), _ptr(old_logp), _ptr(adv),
        _ptr(pi), _ptr(cu_seqlens), _ptr(sel_idx), _ptr(sel_resp), _ptr(n_sel), n_sel_cap,
        _ptr(dloss), _ptr(loss), _ptr(logp), _ptr(lse), _ptr(dHidden), _ptr(dW), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _stream()))


def nat_trace_begin():
    _check(load().nat_trace_begin())


def nat_trace_end():
    """Returns {kind: (milliseconds, launches)} for the tensor-core kernels traced."""
    ms = (ctypes.c_float * len(TRACE_KINDS))()
    cnt = (ctypes.c_int32 * len(TRACE_KINDS))()
    _check(load().nat_trace_end(ms, cnt))
    return {k: (float(ms[i]), int(cnt[i])) for i, k in enumerate(TRACE_KINDS)}


def alloc_workspace(nbytes, device):
    """256-byte aligned scratch (torch's caching allocator aligns to 512 bytes)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def nat_poll_status(workspace):
    """The NAT_DEV_* bits the last loss call left in its workspace (waits for the stream)."""
    word = ctypes.c_uint32(0)
    _check(load().nat_poll_status(_ptr(workspace), _stream(), ctypes.byref(word)))
    return int(word.value)


device_status = nat_poll_status
