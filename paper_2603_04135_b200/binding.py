"""ctypes binding of libdppo.so: same names as include/dppo.h, argument marshalling only.

Array arguments are torch tensors (their device pointer is passed), raw integer addresses, or None
for the nullable ones.  Every function raises DppoError on a non-zero return code.  There is no
fallback: if the library has not been built, importing this module raises.
"""
import ctypes
import os

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libdppo.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError("libdppo.so is not built: run `python -m paper_2603_04135_b200.build` "
                      "(the CUDA library is the only implementation; there is no CPU path)")
lib = ctypes.CDLL(_LIB_PATH)

F32, BF16 = 0, 1
STATUS_OK, STATUS_BAD_LENGTH, STATUS_BAD_TARGET, STATUS_TIMEOUT, STATUS_BAD_SEGMENTS, STATUS_BAD_INDEX, STATUS_RANGE = \
    0, 1, 2, 3, 4, 5, 6
ERR_INVALID_ARG, ERR_BAD_SHAPE, ERR_MISALIGNED, ERR_WORKSPACE_TOO_SMALL, ERR_UNSUPPORTED, ERR_CUDA = \
    -1, -2, -3, -4, -5, -6


class DppoError(RuntimeError):
    def __init__(self, code, message):
        super().__init__("libdppo error %d: %s" % (code, message))
        self.code = code


class PruneParams(ctypes.Structure):
    _fields_ = [("P", ctypes.c_int32), ("G", ctypes.c_int32), ("r_q", ctypes.c_double), ("r_o", ctypes.c_double),
                ("mode", ctypes.c_int32), ("reverse", ctypes.c_int32), ("seed", ctypes.c_uint64),
                ("step", ctypes.c_uint64)]


class PackParams(ctypes.Structure):
    _fields_ = [("n_max", ctypes.c_int32), ("L_row", ctypes.c_int32), ("N_win", ctypes.c_int32),
                ("policy", ctypes.c_int32)]


class LossParams(ctypes.Structure):
    _fields_ = [("T_max", ctypes.c_int64), ("V", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("row_stride", ctypes.c_int64), ("S_max", ctypes.c_int32), ("variant", ctypes.c_int32),
                ("eps_lo", ctypes.c_double), ("eps_hi", ctypes.c_double), ("beta", ctypes.c_double),
                ("temperature", ctypes.c_double), ("no_length_norm", ctypes.c_int32), ("reserved2", ctypes.c_int32),
                ("seq_log_ratio", ctypes.c_void_p)]


class LossKernelChoice(ctypes.Structure):
    _fields_ = [("kernel", ctypes.c_int32), ("ctas_per_row", ctypes.c_int32), ("threads", ctypes.c_int32),
                ("fell_back", ctypes.c_int32)]


KERNEL_GENERAL, KERNEL_WARP, KERNEL_SHARED, KERNEL_STREAM, KERNEL_TILE = 0, 1, 2, 3, 4
KERNEL_NAMES = {KERNEL_GENERAL: "general two-pass", KERNEL_WARP: "warp per row", KERNEL_SHARED: "shared memory",
                KERNEL_STREAM: "streaming (forward only)", KERNEL_TILE: "tiles of rows"}
LOSS_WAIT_SELF_TEST = 1000000      # added to dppo_loss_params.variant
LMHEAD_WAIT_SELF_TEST = 100        # added to dppo_lmhead_params.variant


class LmheadParams(ctypes.Structure):
    _fields_ = [("loss", LossParams), ("H", ctypes.c_int32), ("backward", ctypes.c_int32), ("variant", ctypes.c_int32),
                ("dW_dtype", ctypes.c_int32),
                ("accumulate_dW", ctypes.c_int32), ("reserved", ctypes.c_int32)]


_vp = ctypes.c_void_p
lib.dppo_version.restype = ctypes.c_int
lib.dppo_last_error.restype = ctypes.c_char_p
lib.dppo_group_advantages.restype = ctypes.c_int
lib.dppo_group_advantages.argtypes = [_vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_double, _vp, _vp, _vp, _vp]
lib.dppo_prune_and_rescale.restype = ctypes.c_int
lib.dppo_prune_and_rescale.argtypes = [ctypes.POINTER(PruneParams)] + [_vp] * 17
lib.dppo_history_gather.restype = ctypes.c_int
lib.dppo_history_gather.argtypes = [_vp, ctypes.c_int, _vp, ctypes.c_int, _vp, _vp, _vp]
lib.dppo_history_scatter.restype = ctypes.c_int
lib.dppo_history_scatter.argtypes = [_vp, ctypes.c_int, _vp, ctypes.c_int, _vp, _vp, _vp]
lib.dppo_pack_workspace_bytes.restype = ctypes.c_size_t
lib.dppo_pack_workspace_bytes.argtypes = [ctypes.POINTER(PackParams)]
lib.dppo_pack_prompts.restype = ctypes.c_int
lib.dppo_pack_prompts.argtypes = [ctypes.POINTER(PackParams)] + [_vp] * 10 + [ctypes.c_size_t, _vp, _vp]
lib.dppo_pack_static_max_units.restype = ctypes.c_int
lib.dppo_pack_prompts_static.restype = ctypes.c_int
lib.dppo_pack_prompts_static.argtypes = [ctypes.POINTER(PackParams)] + [_vp] * 11
lib.dppo_grpo_loss_workspace_bytes.restype = ctypes.c_size_t
lib.dppo_grpo_loss_workspace_bytes.argtypes = [ctypes.POINTER(LossParams)]
lib.dppo_grpo_loss_fwd_bwd.restype = ctypes.c_int
lib.dppo_grpo_loss_fwd_bwd.argtypes = [ctypes.POINTER(LossParams)] + [_vp] * 14 + [ctypes.c_size_t, _vp, _vp]


lib.dppo_grpo_loss_kernel_choice.restype = ctypes.c_int
lib.dppo_grpo_loss_kernel_choice.argtypes = [ctypes.POINTER(LossParams), ctypes.c_int, ctypes.POINTER(LossKernelChoice)]
lib.dppo_sequence_log_ratio.restype = ctypes.c_int
lib.dppo_sequence_log_ratio.argtypes = [_vp, _vp, _vp, ctypes.c_int, _vp, _vp, _vp]
lib.dppo_lmhead_workspace_bytes.restype = ctypes.c_size_t
lib.dppo_lmhead_workspace_bytes.argtypes = [ctypes.POINTER(LmheadParams)]
lib.dppo_lmhead_grpo_loss.restype = ctypes.c_int
lib.dppo_lmhead_grpo_loss.argtypes = [ctypes.POINTER(LmheadParams)] + [_vp] * 16 + [ctypes.c_size_t, _vp, _vp]


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, torch.Tensor):
        return x.data_ptr()
    return int(x)


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else None
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream
    return int(stream)


def _check(rc):
    if rc != 0:
        raise DppoError(rc, lib.dppo_last_error().decode("utf-8", "replace"))


def version():
    return lib.dppo_version()


def last_error():
    return lib.dppo_last_error().decode("utf-8", "replace")


def group_advantages(rewards, P, G, adv, mean_abs_adv, std_ddof=0, std_eps=1e-6, status=None, stream=None):
    _check(lib.dppo_group_advantages(_ptr(rewards), P, G, std_ddof, std_eps, _ptr(adv), _ptr(mean_abs_adv),
                                     _ptr(status), _stream(stream)))


def prune_and_rescale(params, adv, mean_abs_adv, H_prev, u_q, u_o, cand_q, cand_o, keep_q, keep_o,
                      n_keep_q, n_keep_o, gamma_q, gamma_o, w_seq, H_next, status=None, stream=None):
    _check(lib.dppo_prune_and_rescale(ctypes.byref(params), _ptr(adv), _ptr(mean_abs_adv), _ptr(H_prev),
                                      _ptr(u_q), _ptr(u_o), _ptr(cand_q), _ptr(cand_o), _ptr(keep_q),
                                      _ptr(keep_o), _ptr(n_keep_q), _ptr(n_keep_o), _ptr(gamma_q),
                                      _ptr(gamma_o), _ptr(w_seq), _ptr(H_next), _ptr(status), _stream(stream)))


def history_gather(H_table, N, prompt_ids, P, H_batch, status=None, stream=None):
    _check(lib.dppo_history_gather(_ptr(H_table), N, _ptr(prompt_ids), P, _ptr(H_batch), _ptr(status), _stream(stream)))


def history_scatter(H_table, N, prompt_ids, P, H_next, status=None, stream=None):
    _check(lib.dppo_history_scatter(_ptr(H_table), N, _ptr(prompt_ids), P, _ptr(H_next), _ptr(status), _stream(stream)))


def pack_workspace_bytes(params):
    return lib.dppo_pack_workspace_bytes(ctypes.byref(params))


def pack_prompts(params, len_, keep, loss_len, order, row_of, off_in_row, row_fill, cu_seqlens, counts,
                 workspace, workspace_bytes, status=None, stream=None):
    _check(lib.dppo_pack_prompts(ctypes.byref(params), _ptr(len_), _ptr(keep), _ptr(loss_len), _ptr(order),
                                 _ptr(row_of), _ptr(off_in_row), _ptr(row_fill), _ptr(cu_seqlens),
                                 _ptr(counts), _ptr(workspace), workspace_bytes, _ptr(status), _stream(stream)))


def pack_static_max_units():
    return lib.dppo_pack_static_max_units()


def pack_prompts_static(params, len_, keep, loss_len, order, row_of, off_in_row, row_fill, cu_seqlens, counts,
                        status=None, stream=None):
    """dppo_pack_prompts without a workspace argument: scratch is a fixed array inside the library
    (at most pack_static_max_units() units); nothing is allocated by the call."""
    _check(lib.dppo_pack_prompts_static(ctypes.byref(params), _ptr(len_), _ptr(keep), _ptr(loss_len), _ptr(order),
                                        _ptr(row_of), _ptr(off_in_row), _ptr(row_fill), _ptr(cu_seqlens),
                                        _ptr(counts), _ptr(status), _stream(stream)))


def grpo_loss_workspace_bytes(params):
    return lib.dppo_grpo_loss_workspace_bytes(ctypes.byref(params))


def grpo_loss_fwd_bwd(params, logits, target, logp_old, logp_ref, cu_seqlens, n_tokens_dev, adv, w, seg_map,
                      dlogits, logp_out, lse_out, loss_out, workspace, workspace_bytes, status=None,
                      stream=None):
    _check(lib.dppo_grpo_loss_fwd_bwd(ctypes.byref(params), _ptr(logits), _ptr(target), _ptr(logp_old),
                                      _ptr(logp_ref), _ptr(cu_seqlens), _ptr(n_tokens_dev), _ptr(adv), _ptr(w),
                                      _ptr(seg_map), _ptr(dlogits), _ptr(logp_out), _ptr(lse_out),
                                      _ptr(loss_out), _ptr(workspace), workspace_bytes, _ptr(status),
                                      _stream(stream)))


def grpo_loss_kernel_choice(params, forward_only=False):
    """The kernel dppo_grpo_loss_fwd_bwd runs for these parameters on the current device (forward_only: the call
    will pass no dlogits), as a LossKernelChoice."""
    out = LossKernelChoice()
    _check(lib.dppo_grpo_loss_kernel_choice(ctypes.byref(params), int(bool(forward_only)), ctypes.byref(out)))
    return out


def lmhead_workspace_bytes(params):
    return lib.dppo_lmhead_workspace_bytes(ctypes.byref(params))


def lmhead_grpo_loss(params, hidden, W, target, logp_old, logp_ref, cu_seqlens, n_tokens_dev, adv, w, seg_map,
                     dhidden, dW, logp_out, lse_out, loss_out, workspace, workspace_bytes, status=None, stream=None):
    _check(lib.dppo_lmhead_grpo_loss(ctypes.byref(params), _ptr(hidden), _ptr(W), _ptr(target), _ptr(logp_old),
                                     _ptr(logp_ref), _ptr(cu_seqlens), _ptr(n_tokens_dev), _ptr(adv), _ptr(w),
                                     _ptr(seg_map), _ptr(dhidden), _ptr(dW), _ptr(logp_out), _ptr(lse_out),
                                     _ptr(loss_out), _ptr(workspace), workspace_bytes, _ptr(status), _stream(stream)))


def sequence_log_ratio(logp, logp_old, cu_seqlens, S_max, out, status=None, stream=None):
    _check(lib.dppo_sequence_log_ratio(_ptr(logp), _ptr(logp_old), _ptr(cu_seqlens), S_max, _ptr(out), _ptr(status),
                                       _stream(stream)))
