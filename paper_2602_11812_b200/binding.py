"""ctypes binding of libegtp_b200.so: the same entry points as include/egtp.h, argument marshalling only.

Every step of the path runs in the library's CUDA kernels; torch is used for device memory
and streams.  Loading fails loudly when the library has not been built
(`python -m paper_2602_11812_b200.build`); there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

LIB_NAME = "libegtp_b200.so"
LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), LIB_NAME)

EGTP_OK = 0
EGTP_ERR_INVALID_ARG = -1
EGTP_ERR_UNSUPPORTED = -2
EGTP_ERR_CAPACITY = -3
EGTP_ERR_CUDA = -4
EGTP_ERR_BAD_OFFSETS = -5
EGTP_ERR_DEVICE_TIMEOUT = -6
EGTP_ERR_BAD_SLOT = -7
EGTP_F32, EGTP_BF16 = 0, 1
EGTP_HEAD_SCALAR, EGTP_HEAD_BINS = 0, 1
PLP_RESET_KEEP, PLP_RESET_EMPTY = -2, -1
EGTP_LMHEAD_AUTO, EGTP_LMHEAD_CTA_PAIRS, EGTP_LMHEAD_SINGLE_CTA, EGTP_LMHEAD_CTA_PAIRS_WIDE = 0, 1, 2, 3
EGTP_POOL_MEAN, EGTP_POOL_MAX, EGTP_POOL_LAST = 1, 2, 3
EGTP_CREATE_NO_HOST_STAGING = 1
KERNEL_IDS = ["validate_offsets", "lmhead_entropy", "entropy_merge", "token_weights", "pool",
              "pool_combine", "head_hidden", "head_out", "plp_update", "logits_entropy", "stage_rows"]
EGTP_NUM_KERNELS = len(KERNEL_IDS)
EGTP_K_LMHEAD_ENTROPY = 1

EXPORTED_SYMBOLS = [
    "egtp_create", "egtp_destroy", "egtp_status_string", "egtp_workspace_bytes", "egtp_predict",
    "egtp_predict_host", "plp_state_create", "plp_state_destroy", "plp_state_export", "plp_state_import",
    "plp_step", "plp_step_host", "egtp_profile_enable", "egtp_profile_read", "egtp_kernel_name",
    "egtp_launch_count", "egtp_lmhead_plan", "egtp_head_forward_static", "egtp_set_lmhead_mode",
    "egtp_entropy_from_logits", "plp_step_from_logits", "egtp_pool_baseline",
    "egtp_entropy_partials", "egtp_entropy_from_partials", "plp_step_from_partials", "egtp_selftest_wait_timeout",
    "plp_state_bind_head", "egtp_set_lmhead_chunks", "egtp_lmhead_plan_for", "egtp_create_ex", "egtp_set_launch_overlap", "plp_step_host_async",
]


class egtp_lm_head(C.Structure):
    _fields_ = [("W", C.c_void_p), ("ldw", C.c_int64), ("d", C.c_int32), ("V", C.c_int32),
                ("dtype", C.c_int32), ("reserved", C.c_int32)]


class egtp_head(C.Structure):
    _fields_ = [("W1", C.c_void_p), ("b1", C.c_void_p), ("W2", C.c_void_p), ("b2", C.c_void_p),
                ("centres", C.c_void_p), ("d", C.c_int32), ("m_h", C.c_int32), ("d_out", C.c_int32),
                ("wdtype", C.c_int32), ("mode", C.c_int32), ("reserved", C.c_int32)]


class EgtpError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


_lib = None


def load() -> C.CDLL:
    """Loads the shared library (once) and declares every prototype of include/egtp.h."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_11812_b200.build` "
                          "(there is no CPU or library fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
    P = C.POINTER
    lib.egtp_create.argtypes = [P(vp), C.c_int, i64, i32, i32, i32]
    lib.egtp_create_ex.argtypes = [P(vp), C.c_int, i64, i32, i32, i32, i32]
    lib.egtp_destroy.argtypes = [vp]
    lib.egtp_status_string.argtypes = [C.c_int]
    lib.egtp_status_string.restype = C.c_char_p
    lib.egtp_kernel_name.argtypes = [C.c_int]
    lib.egtp_kernel_name.restype = C.c_char_p
    lib.egtp_workspace_bytes.argtypes = [vp]
    lib.egtp_workspace_bytes.restype = i64
    lib.egtp_launch_count.argtypes = [vp]
    lib.egtp_launch_count.restype = i64
    lib.egtp_lmhead_plan.argtypes = [vp, i64, i32, i32, i32, P(i32)]
    lib.egtp_profile_enable.argtypes = [vp, C.c_int]
    lib.egtp_set_lmhead_mode.argtypes = [vp, C.c_int]
    lib.egtp_set_lmhead_chunks.argtypes = [vp, i32]
    lib.egtp_set_launch_overlap.argtypes = [vp, C.c_int]
    lib.egtp_lmhead_plan_for.argtypes = [i32, i32, i64, i32, i32, i32, i32, i32, P(i32)]
    lib.egtp_selftest_wait_timeout.argtypes = [vp, i32, vp, vp]
    lib.egtp_entropy_partials.argtypes = [vp, P(egtp_lm_head), vp, i64, i64, vp, vp, vp]
    lib.egtp_entropy_from_partials.argtypes = [vp, vp, i32, i64, vp, vp, vp]
    lib.plp_step_from_partials.argtypes = [vp, vp, vp, i32, P(egtp_head), vp, i64, i32, vp, vp, vp, vp, vp, i32, i32, f32,
                                           vp, vp, vp, vp, vp]
    lib.egtp_pool_baseline.argtypes = [vp, P(egtp_head), vp, i64, i32, i32, vp, i32, i64, i32, vp, vp, vp, vp]
    lib.egtp_entropy_from_logits.argtypes = [vp, vp, i64, i32, i64, i32, vp, vp, vp]
    lib.plp_step_from_logits.argtypes = [vp, vp, vp, i64, i32, i32, P(egtp_head), vp, i64, i32, vp, vp, vp, vp, vp, i32, i32,
                                         f32, vp, vp, vp, vp, vp]
    lib.egtp_profile_read.argtypes = [vp, P(C.c_double), P(i64)]
    lib.egtp_predict.argtypes = [vp, P(egtp_lm_head), P(egtp_head), vp, i64, vp, i32, i64, f32,
                                 vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.egtp_predict_host.argtypes = [vp, P(egtp_lm_head), P(egtp_head), vp, vp, i32, i64, f32, vp, vp, vp, vp]
    lib.plp_state_create.argtypes = [vp, P(vp), i32, i32]
    lib.plp_state_destroy.argtypes = [vp]
    lib.plp_state_export.argtypes = [vp, vp, vp, vp, vp]
    lib.plp_state_import.argtypes = [vp, vp, vp, vp, vp]
    lib.plp_state_bind_head.argtypes = [vp, P(egtp_head)]
    lib.plp_step.argtypes = [vp, vp, P(egtp_lm_head), P(egtp_head), vp, i64, vp, vp, vp, vp, vp, i32, i32, f32,
                             vp, vp, vp, vp, vp]
    lib.plp_step_host.argtypes = [vp, vp, P(egtp_lm_head), P(egtp_head), vp, vp, vp, vp, vp, i32, i32, f32,
                                  vp, vp, vp]
    lib.plp_step_host_async.argtypes = lib.plp_step_host.argtypes
    lib.egtp_head_forward_static.argtypes = [P(egtp_head), vp, i64, i32, vp, vp, vp]
    for name in EXPORTED_SYMBOLS:
        fn = getattr(lib, name)
        if name not in ("egtp_status_string", "egtp_kernel_name", "egtp_workspace_bytes", "egtp_launch_count"):
            fn.restype = C.c_int
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().egtp_status_string(int(status)).decode()


def _check(rc: int, where: str):
    if rc != EGTP_OK:
        raise EgtpError(rc, where)


def _ptr(t) -> Optional[int]:
    """Device (or host) address of a torch tensor / numpy array, None for None."""
    if t is None:
        return None
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    if hasattr(stream, "cuda_stream"):
        return stream.cuda_stream or None
    return int(stream) or None


def _dtype_code(t) -> int:
    import torch
    if t.dtype == torch.bfloat16:
        return EGTP_BF16
    if t.dtype == torch.float32:
        return EGTP_F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def make_lm_head(W) -> egtp_lm_head:
    """W: device tensor [V, d] (row-major, possibly with a row stride)."""
    assert W.is_cuda and W.dim() == 2 and W.stride(1) == 1
    return egtp_lm_head(W=W.data_ptr(), ldw=W.stride(0), d=W.shape[1], V=W.shape[0], dtype=_dtype_code(W), reserved=0)


def make_head(W1, b1, W2, b2, mode: int = EGTP_HEAD_SCALAR, centres=None) -> egtp_head:
    """W1 [m_h, d], W2 [d_out, m_h] contiguous device tensors of one dtype; b1, b2, centres float32."""
    import torch
    assert W1.is_contiguous() and W2.is_contiguous() and W1.dtype == W2.dtype
    assert b1.dtype == torch.float32 and b2.dtype == torch.float32
    return egtp_head(W1=W1.data_ptr(), b1=b1.data_ptr(), W2=W2.data_ptr(), b2=b2.data_ptr(),
                     centres=None if centres is None else centres.data_ptr(), d=W1.shape[1], m_h=W1.shape[0],
                     d_out=W2.shape[0], wdtype=_dtype_code(W1), mode=mode, reserved=0)


# --------------------------------------------------------------------------- entry points
def egtp_create(device: int, max_tokens: int, max_batch: int, max_d: int, max_V: int) -> int:
    ctx = C.c_void_p()
    _check(load().egtp_create(C.byref(ctx), device, max_tokens, max_batch, max_d, max_V), "egtp_create")
    return ctx.value


def egtp_create_ex(device: int, max_tokens: int, max_batch: int, max_d: int, max_V: int, flags: int = 0,
                   check: bool = True):
    """egtp_create with option flags (EGTP_CREATE_NO_HOST_STAGING); returns the context handle (or the status with check=False)."""
    ctx = C.c_void_p()
    rc = load().egtp_create_ex(C.byref(ctx), device, max_tokens, max_batch, max_d, max_V, flags)
    if check:
        _check(rc, "egtp_create_ex")
        return ctx.value
    return rc


def egtp_destroy(ctx: int):
    _check(load().egtp_destroy(ctx), "egtp_destroy")


def egtp_workspace_bytes(ctx: int) -> int:
    return load().egtp_workspace_bytes(ctx)


def egtp_launch_count(ctx: int) -> int:
    return load().egtp_launch_count(ctx)


def egtp_kernel_name(kernel_id: int) -> str:
    return load().egtp_kernel_name(kernel_id).decode()


def egtp_lmhead_plan(ctx: int, T: int, d: int, V: int, dtype: int) -> dict:
    info = (C.c_int32 * 8)()
    _check(load().egtp_lmhead_plan(ctx, T, d, V, dtype, info), "egtp_lmhead_plan")
    keys = ["grid", "row_blocks", "rows_per_block", "chunks", "slots", "tile_cols", "k_blocks", "smem_bytes"]
    return dict(zip(keys, list(info)))


def egtp_lmhead_plan_for(num_sms: int, pair_workers: int, T: int, d: int, V: int, dtype: int = EGTP_BF16,
                         mode: int = EGTP_LMHEAD_AUTO, head_cols: int = 0) -> dict:
    """Launch plan of the LM-head kernel for a device described by its SM count (no GPU needed)."""
    info = (C.c_int32 * 12)()
    _check(load().egtp_lmhead_plan_for(num_sms, pair_workers, T, d, V, dtype, mode, head_cols, info), "egtp_lmhead_plan_for")
    keys = ["grid", "row_blocks", "rows_per_block", "chunks", "slots", "tile_cols", "k_blocks", "smem_bytes",
            "variant", "group_rb", "col_gran", "n_groups"]
    return dict(zip(keys, list(info)))


def egtp_set_lmhead_mode(ctx: int, mode: int):
    _check(load().egtp_set_lmhead_mode(ctx, mode), "egtp_set_lmhead_mode")


def egtp_set_lmhead_chunks(ctx: int, chunks: int):
    """Forces the number of vocabulary chunks of prompt batches (0 = chosen by the library)."""
    _check(load().egtp_set_lmhead_chunks(ctx, chunks), "egtp_set_lmhead_chunks")


def egtp_set_launch_overlap(ctx: int, on: bool):
    _check(load().egtp_set_launch_overlap(ctx, 1 if on else 0), "egtp_set_launch_overlap")


def egtp_profile_enable(ctx: int, on: bool):
    _check(load().egtp_profile_enable(ctx, 1 if on else 0), "egtp_profile_enable")


def egtp_profile_read(ctx: int) -> dict:
    ms = (C.c_double * EGTP_NUM_KERNELS)()
    n = (C.c_int64 * EGTP_NUM_KERNELS)()
    _check(load().egtp_profile_read(ctx, ms, n), "egtp_profile_read")
    return {KERNEL_IDS[k]: dict(ms=ms[k], launches=n[k]) for k in range(EGTP_NUM_KERNELS)}


def egtp_predict(ctx: int, lm: egtp_lm_head, head: Optional[egtp_head], hidden, offsets, B: int, T_total: int,
                 alpha: float = 1.0, H_out=None, weights_out=None, seg_id_out=None, pooled_out=None,
                 state_m_out=None, state_s_out=None, yhat_out=None, phat_out=None, status_dev=None, stream=None,
                 ldh: Optional[int] = None, check: bool = True) -> int:
    if ldh is None:
        ldh = hidden.stride(0) if hidden is not None and hasattr(hidden, "stride") else lm.d
    rc = load().egtp_predict(ctx, C.byref(lm), C.byref(head) if head is not None else None, _ptr(hidden), ldh,
                             _ptr(offsets), B, T_total, alpha, _ptr(H_out), _ptr(weights_out), _ptr(seg_id_out),
                             _ptr(pooled_out), _ptr(state_m_out), _ptr(state_s_out), _ptr(yhat_out), _ptr(phat_out),
                             _ptr(status_dev), _stream(stream))
    if check:
        _check(rc, "egtp_predict")
    return rc


def egtp_predict_host(ctx: int, lm: egtp_lm_head, head: egtp_head, hidden_host, offsets_host, B: int, T_total: int,
                      alpha: float, yhat_host, pooled_host, status_host, stream=None, check: bool = True) -> int:
    rc = load().egtp_predict_host(ctx, C.byref(lm), C.byref(head), _ptr(hidden_host), _ptr(offsets_host), B, T_total,
                                  alpha, _ptr(yhat_host), _ptr(pooled_host), _ptr(status_host), _stream(stream))
    if check:
        _check(rc, "egtp_predict_host")
    return rc


def plp_state_create(ctx: int, num_slots: int, d: int) -> int:
    st = C.c_void_p()
    _check(load().plp_state_create(ctx, C.byref(st), num_slots, d), "plp_state_create")
    return st.value


def plp_state_destroy(st: int):
    _check(load().plp_state_destroy(st), "plp_state_destroy")


def plp_state_export(st: int, m, s, acc, stream=None):
    _check(load().plp_state_export(st, _ptr(m), _ptr(s), _ptr(acc), _stream(stream)), "plp_state_export")


def plp_state_import(st: int, m, s, acc, stream=None):
    _check(load().plp_state_import(st, _ptr(m), _ptr(s), _ptr(acc), _stream(stream)), "plp_state_import")


def plp_state_bind_head(st: int, head: egtp_head, check: bool = True) -> int:
    """Fixes the head a PLP state is used with: plp_step then gets W1 h' from the LM-head kernel itself."""
    rc = load().plp_state_bind_head(st, C.byref(head))
    if check:
        _check(rc, "plp_state_bind_head")
    return rc


def plp_step(ctx: int, st: int, lm: egtp_lm_head, head: Optional[egtp_head], hidden_step, slot_ids=None,
             reset_src=None, src_m=None, src_s=None, src_pooled=None, n_src: int = 0, B_live: Optional[int] = None,
             alpha: float = 1.0, Hstep_out=None, z_out=None, yrem_out=None, status_dev=None, stream=None,
             ldh: Optional[int] = None, check: bool = True) -> int:
    if B_live is None:
        B_live = hidden_step.shape[0]
    if ldh is None:
        ldh = hidden_step.stride(0) if hasattr(hidden_step, "stride") else lm.d
    rc = load().plp_step(ctx, st, C.byref(lm), C.byref(head) if head is not None else None, _ptr(hidden_step), ldh,
                         _ptr(slot_ids), _ptr(reset_src), _ptr(src_m), _ptr(src_s), _ptr(src_pooled), n_src, B_live,
                         alpha, _ptr(Hstep_out), _ptr(z_out), _ptr(yrem_out), _ptr(status_dev), _stream(stream))
    if check:
        _check(rc, "plp_step")
    return rc


def plp_step_host(ctx: int, st: int, lm: egtp_lm_head, head: egtp_head, hidden_step_host, reset_src_host,
                  src_m, src_s, src_pooled, n_src: int, B_live: int, alpha: float, yrem_host, status_host,
                  stream=None, check: bool = True) -> int:
    rc = load().plp_step_host(ctx, st, C.byref(lm), C.byref(head), _ptr(hidden_step_host), _ptr(reset_src_host),
                              _ptr(src_m), _ptr(src_s), _ptr(src_pooled), n_src, B_live, alpha, _ptr(yrem_host),
                              _ptr(status_host), _stream(stream))
    if check:
        _check(rc, "plp_step_host")
    return rc


def plp_step_host_async(ctx: int, st: int, lm: egtp_lm_head, head: egtp_head, hidden_step_host, reset_src_host,
                        src_m, src_s, src_pooled, n_src: int, B_live: int, alpha: float, yrem_host, status_host,
                        stream=None, check: bool = True) -> int:
    """plp_step_host without the final wait: results are in yrem_host / status_host once the stream has caught up."""
    rc = load().plp_step_host_async(ctx, st, C.byref(lm), C.byref(head), _ptr(hidden_step_host), _ptr(reset_src_host),
                                    _ptr(src_m), _ptr(src_s), _ptr(src_pooled), n_src, B_live, alpha, _ptr(yrem_host),
                                    _ptr(status_host), _stream(stream))
    if check:
        _check(rc, "plp_step_host_async")
    return rc


def egtp_head_forward_static(head: egtp_head, z, rows: Optional[int] = None, y_out=None, phat_out=None, stream=None,
                             ldz: Optional[int] = None, check: bool = True) -> int:
    """Head forward pass without a context and without any device allocation (fixed in-library scratch).

    For callers that may not allocate GPU memory; rows * m_h is limited to 2**20.  Calls on one
    device share the scratch, so they must not overlap on the GPU.
    """
    if rows is None:
        rows = z.shape[0]
    if ldz is None:
        ldz = z.stride(0) if hasattr(z, "stride") else head.d
    rc = load().egtp_head_forward_static(C.byref(head), _ptr(z), ldz, rows, _ptr(y_out), _ptr(phat_out),
                                         _stream(stream))
    if check:
        _check(rc, "egtp_head_forward_static")
    return rc


def egtp_entropy_from_logits(ctx: int, logits, H_out, rows: Optional[int] = None, V: Optional[int] = None,
                             status_dev=None, stream=None, check: bool = True) -> int:
    """H_out[i] = entropy of softmax(logits[i]) for a device tensor logits [rows, V] (bf16 or fp32)."""
    rows = logits.shape[0] if rows is None else rows
    V = logits.shape[1] if V is None else V
    rc = load().egtp_entropy_from_logits(ctx, _ptr(logits), logits.stride(0), _dtype_code(logits), rows, V,
                                         _ptr(H_out), _ptr(status_dev), _stream(stream))
    if check:
        _check(rc, "egtp_entropy_from_logits")
    return rc


def plp_step_from_logits(ctx: int, st: int, logits, head: Optional[egtp_head], hidden_step, slot_ids=None,
                         reset_src=None, src_m=None, src_s=None, src_pooled=None, n_src: int = 0,
                         B_live: Optional[int] = None, alpha: float = 1.0, Hstep_out=None, z_out=None, yrem_out=None,
                         status_dev=None, stream=None, check: bool = True) -> int:
    """plp_step with the step's entropies computed from logits [B_live, V] that are already in device memory."""
    if B_live is None:
        B_live = hidden_step.shape[0]
    rc = load().plp_step_from_logits(ctx, st, _ptr(logits), logits.stride(0), _dtype_code(logits), logits.shape[1],
                                     C.byref(head) if head is not None else None, _ptr(hidden_step),
                                     hidden_step.stride(0), _dtype_code(hidden_step), _ptr(slot_ids), _ptr(reset_src),
                                     _ptr(src_m), _ptr(src_s), _ptr(src_pooled), n_src, B_live, alpha,
                                     _ptr(Hstep_out), _ptr(z_out), _ptr(yrem_out), _ptr(status_dev), _stream(stream))
    if check:
        _check(rc, "plp_step_from_logits")
    return rc


def egtp_pool_baseline(ctx: int, head: Optional[egtp_head], hidden, offsets, B: int, T_total: int, mode: int,
                       pooled_out=None, yhat_out=None, status_dev=None, stream=None, check: bool = True) -> int:
    """Average / max / last-token pooling (the paper's ablation comparators) over a ragged batch, then the head."""
    rc = load().egtp_pool_baseline(ctx, C.byref(head) if head is not None else None, _ptr(hidden), hidden.stride(0),
                                   _dtype_code(hidden), hidden.shape[1], _ptr(offsets), B, T_total, mode,
                                   _ptr(pooled_out), _ptr(yhat_out), _ptr(status_dev), _stream(stream))
    if check:
        _check(rc, "egtp_pool_baseline")
    return rc


def egtp_entropy_partials(ctx: int, lm_shard: egtp_lm_head, hidden, partial_out, rows: Optional[int] = None,
                          status_dev=None, stream=None, check: bool = True) -> int:
    """(m, s, t2) per row over this GPU's shard of the vocabulary; partial_out float32 [rows, 3]."""
    rows = hidden.shape[0] if rows is None else rows
    rc = load().egtp_entropy_partials(ctx, C.byref(lm_shard), _ptr(hidden), hidden.stride(0), rows, _ptr(partial_out),
                                      _ptr(status_dev), _stream(stream))
    if check:
        _check(rc, "egtp_entropy_partials")
    return rc


def egtp_entropy_from_partials(ctx: int, gathered, H_out, status_dev=None, stream=None, check: bool = True) -> int:
    """gathered float32 [num_shards, rows, 3] (rank-major, as an all-gather leaves it) -> H_out [rows]."""
    rc = load().egtp_entropy_from_partials(ctx, _ptr(gathered), gathered.shape[0], gathered.shape[1], _ptr(H_out),
                                           _ptr(status_dev), _stream(stream))
    if check:
        _check(rc, "egtp_entropy_from_partials")
    return rc


def plp_step_from_partials(ctx: int, st: int, gathered, head: Optional[egtp_head], hidden_step, slot_ids=None,
                           reset_src=None, src_m=None, src_s=None, src_pooled=None, n_src: int = 0,
                           alpha: float = 1.0, Hstep_out=None, z_out=None, yrem_out=None, status_dev=None, stream=None,
                           check: bool = True) -> int:
    """plp_step with the step's entropies merged from vocabulary-shard triples gathered [num_shards, B_live, 3]."""
    rc = load().plp_step_from_partials(ctx, st, _ptr(gathered), gathered.shape[0], C.byref(head) if head is not None else None,
                                       _ptr(hidden_step), hidden_step.stride(0), _dtype_code(hidden_step), _ptr(slot_ids),
                                       _ptr(reset_src), _ptr(src_m), _ptr(src_s), _ptr(src_pooled), n_src,
                                       gathered.shape[1], alpha, _ptr(Hstep_out), _ptr(z_out), _ptr(yrem_out),
                                       _ptr(status_dev), _stream(stream))
    if check:
        _check(rc, "plp_step_from_partials")
    return rc


def egtp_selftest_wait_timeout(ctx: int, limit_ms: int, status_dev, stream=None, check: bool = True) -> int:
    """Runs a bounded wait that nothing will satisfy; status_dev ends up holding EGTP_ERR_DEVICE_TIMEOUT."""
    rc = load().egtp_selftest_wait_timeout(ctx, limit_ms, _ptr(status_dev), _stream(stream))
    if check:
        _check(rc, "egtp_selftest_wait_timeout")
    return rc
