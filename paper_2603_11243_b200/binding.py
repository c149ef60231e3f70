"""Thin Python binding of libssd's C ABI (argument marshalling only).

Every function here takes torch tensors that already live on the CUDA device, passes their
addresses to the C entry point of the same name and returns the output tensors; all
computation happens in the library's CUDA kernels.  There is no CPU fallback: importing this
module without a built libssd.so, or calling it with host tensors, raises.
"""
import ctypes as C
import os
from typing import Callable, Dict, List, Optional

import torch

F32, BF16 = 0, 1
UTT_NONFINITE, UTT_BAD_DRAFT_ID, UTT_BAD_OFFSETS, UTT_INTERNAL = 1, 2, 4, 0x80000000
OK, ERR_NULL, ERR_ARG, ERR_DTYPE, ERR_WORKSPACE, ERR_CUDA, ERR_ALIGN, ERR_TOO_LARGE = range(8)
VERIFY_STATIC_SCRATCH_BYTES = 8 << 20

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libssd.so")


class SsdError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().ssd_status_string(code).decode()
        if code == ERR_CUDA:
            msg += " (cudaError %d)" % lib().ssd_last_cuda_error()
        super().__init__("%s: %s" % (where, msg))


class LaunchOpts(C.Structure):
    """Mirror of ssd_launch_opts (include/ssd.h)."""
    _fields_ = [("kernel", C.c_int32), ("ctas", C.c_int32), ("warps", C.c_int32),
                ("stages", C.c_int32), ("stage_bytes", C.c_int32), ("split", C.c_int32),
                ("ev_begin", C.c_void_p), ("ev_end", C.c_void_p), ("fma_exp", C.c_int32),
                ("finish", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                "libssd.so is not built: run `python -m paper_2603_11243_b200.build` "
                "(needs nvcc); there is no fallback path")
        L = C.CDLL(LIB_PATH)
        L.ssd_status_string.restype = C.c_char_p
        L.ssd_status_string.argtypes = [C.c_int32]
        L.ssd_last_cuda_error.restype = C.c_int32
        L.ssd_version.restype = C.c_int32
        L.ssd_launch_count.restype = C.c_uint64
        for f in (L.ssd_ctc_draft_workspace_bytes, L.ssd_verify_workspace_bytes):
            f.restype = C.c_size_t
            f.argtypes = [C.c_int32, C.c_int64, C.c_int32, C.c_int, C.c_void_p]
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        L.ssd_ctc_draft.restype = i32
        L.ssd_ctc_draft.argtypes = [vp, C.c_int, i32, i64, vp, i32, i64, i32, i32,
                                    vp, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                    vp, C.c_size_t, vp, vp]
        L.ssd_entropy_gate.restype = i32
        L.ssd_entropy_gate.argtypes = [vp, vp, i32, i64, C.c_float, vp, vp, vp, vp, vp, vp]
        L.ssd_verify.restype = i32
        L.ssd_verify.argtypes = [vp, C.c_int, i32, i64, vp, vp, i32, i64, C.c_float, vp,
                                 vp, vp, vp, vp, vp, vp, C.c_size_t, vp, vp]
        L.ssd_verify_static.restype = i32
        L.ssd_verify_static.argtypes = [vp, C.c_int, i32, i64, vp, vp, i32, i64, C.c_float, vp,
                                        vp, vp, vp, vp, vp, vp, vp]
        L.ssd_verify_early_exit_workspace_bytes.restype = C.c_size_t
        L.ssd_verify_early_exit_workspace_bytes.argtypes = [C.c_int32, C.c_int64, C.c_int32, C.c_int, C.c_void_p]
        L.ssd_verify_early_exit.restype = i32
        L.ssd_verify_early_exit.argtypes = [vp, C.c_int, i32, i64, vp, vp, i32, i64, C.c_float, vp,
                                            vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp, vp]
        for f in (L.ssd_ctc_draft_read_span, L.ssd_verify_read_span):
            f.restype = i32
        L.ssd_ctc_draft_read_span.argtypes = [C.c_uint64, C.c_int, i32, i64, i64, vp, vp]
        L.ssd_verify_read_span.argtypes = [C.c_uint64, C.c_int, i32, i64, i64, i32, vp, vp]
        L.ssd_verify_shard.restype = i32
        L.ssd_verify_shard.argtypes = [vp, C.c_int, i32, i64, i64, vp, vp, i32, i64, vp, vp, vp,
                                       C.c_size_t, vp, vp]
        L.ssd_verify_combine.restype = i32
        L.ssd_verify_combine.argtypes = [vp, i32, i64, vp, vp, i32, i64, C.c_float, vp, vp, vp, vp,
                                         vp, vp, vp]
        L.ssd_threshold_sweep.restype = i32
        L.ssd_threshold_sweep.argtypes = [vp, vp, vp, i32, i64, vp, vp, i32, vp, vp, vp, vp, vp]
        L.ssd_assemble.restype = i32
        L.ssd_assemble.argtypes = [vp, vp, i32, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.ssd_greedy_step_workspace_bytes.restype = C.c_size_t
        L.ssd_greedy_step_workspace_bytes.argtypes = [i64, i32, C.c_int, vp]
        L.ssd_greedy_step.restype = i32
        L.ssd_greedy_step.argtypes = [vp, C.c_int, i32, i64, i64, vp, vp, vp, vp, vp, C.c_size_t,
                                      vp, vp]
        _lib = L
    return _lib


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("logits must be float32 or bfloat16, got %s" % t.dtype)


def _dev(t: Optional[torch.Tensor], name: str):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor: libssd has no host path" % name)
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _opts(o: Optional[LaunchOpts]):
    return None if o is None else C.cast(C.pointer(o), C.c_void_p)


def _rows_ld(logits: torch.Tensor):
    if logits.dim() != 2 or logits.stride(1) != 1:
        raise ValueError("logits must be a 2-D row-major matrix (unit stride along the vocabulary)")
    return logits.shape[0], (logits.stride(0) if logits.shape[0] > 1 else max(logits.stride(0), logits.shape[1]))


def ssd_ctc_draft_workspace_bytes(B, N, V, dtype_code, opts=None) -> int:
    return int(lib().ssd_ctc_draft_workspace_bytes(B, N, V, dtype_code, _opts(opts)))


def ssd_verify_workspace_bytes(B, M, V, dtype_code, opts=None) -> int:
    return int(lib().ssd_verify_workspace_bytes(B, M, V, dtype_code, _opts(opts)))


class ReadSpan(C.Structure):
    """Mirror of ssd_read_span (include/ssd.h)."""
    _fields_ = [("lo", C.c_uint64), ("hi", C.c_uint64), ("faults", C.c_int64),
                ("kernel", C.c_int32), ("reserved", C.c_int32)]


def ssd_ctc_draft_read_span(base_addr: int, dtype_code: int, V: int, ld: int, N: int,
                            opts: Optional[LaunchOpts] = None) -> ReadSpan:
    """Host-only: the addresses ssd_ctc_draft's streaming kernel would read (see ssd.h)."""
    out = ReadSpan()
    rc = lib().ssd_ctc_draft_read_span(base_addr, dtype_code, V, ld, N, _opts(opts),
                                       C.cast(C.pointer(out), C.c_void_p))
    if rc != OK:
        raise SsdError(rc, "ssd_ctc_draft_read_span")
    return out


def ssd_verify_read_span(base_addr: int, dtype_code: int, V: int, ld: int, M: int, B: int = 1,
                         opts: Optional[LaunchOpts] = None) -> ReadSpan:
    """Host-only: the addresses ssd_verify's streaming kernel would read (see ssd.h)."""
    out = ReadSpan()
    rc = lib().ssd_verify_read_span(base_addr, dtype_code, V, ld, M, B, _opts(opts),
                                    C.cast(C.pointer(out), C.c_void_p))
    if rc != OK:
        raise SsdError(rc, "ssd_verify_read_span")
    return out


def alloc_ctc_outputs(N: int, B: int, device, logprob_ld: int = 0) -> Dict[str, torch.Tensor]:
    e = lambda n, dt: torch.empty((n,), dtype=dt, device=device)
    # ssd_ctc_draft_workspace_bytes is 2048 whatever the sizes are (the tile counters)
    out = dict(workspace=torch.empty((2048,), dtype=torch.uint8, device=device),
               frame_entropy=e(N, torch.float32), frame_argmax=e(N, torch.int32),
               frame_lse=e(N, torch.float32), draft_tokens=e(N, torch.int32),
               draft_frames=e(N, torch.int32), draft_len=e(B, torch.int32),
               draft_full_len=e(B, torch.int32), utt_max_entropy=e(B, torch.float32),
               utt_status=e(B, torch.int32))
    if logprob_ld:
        out["frame_logprob"] = torch.empty((N, logprob_ld), dtype=torch.float32, device=device)
    return out


def ssd_ctc_draft(logits: torch.Tensor, frame_off: torch.Tensor, blank_id: int,
                  max_draft_len: int, V: Optional[int] = None, out=None, want_logprob=False,
                  opts: Optional[LaunchOpts] = None) -> Dict[str, torch.Tensor]:
    """Stage 1 (Section 2.1, Eq. 2, Eq. 3): frame statistics and the collapsed draft."""
    N, ld = _rows_ld(logits)
    V = logits.shape[1] if V is None else V
    B = frame_off.shape[0] - 1
    if frame_off.dtype != torch.int64:
        raise TypeError("frame_off must be int64")
    if out is None:
        out = alloc_ctc_outputs(N, B, logits.device, ld if want_logprob else 0)
    ws = out.get("workspace")
    rc = lib().ssd_ctc_draft(
        _dev(logits, "logits"), _dtype_code(logits), V, ld, _dev(frame_off, "frame_off"), B, N,
        blank_id, max_draft_len, _dev(out["frame_entropy"], "frame_entropy"),
        _dev(out["frame_argmax"], "frame_argmax"), _dev(out.get("frame_lse"), "frame_lse"),
        _dev(out.get("frame_logprob"), "frame_logprob"),
        _dev(out["draft_tokens"], "draft_tokens"), _dev(out.get("draft_frames"), "draft_frames"),
        _dev(out["draft_len"], "draft_len"), _dev(out["draft_full_len"], "draft_full_len"),
        _dev(out["utt_max_entropy"], "utt_max_entropy"), _dev(out["utt_status"], "utt_status"),
        _dev(ws, "workspace"), 0 if ws is None else ws.numel(), _stream(), _opts(opts))
    if rc != OK:
        raise SsdError(rc, "ssd_ctc_draft")
    return out


def alloc_gate_outputs(B: int, device) -> Dict[str, torch.Tensor]:
    return dict(gate_accept=torch.empty((B,), dtype=torch.uint8, device=device),
                max_entropy=torch.empty((B,), dtype=torch.float32, device=device),
                argmax_frame=torch.empty((B,), dtype=torch.int32, device=device))


def ssd_entropy_gate(frame_entropy: torch.Tensor, frame_off: torch.Tensor, tau_ctc: float,
                     out=None) -> Dict[str, torch.Tensor]:
    """The entropy gate (Eq. 3): accept iff every frame entropy is below tau_ctc."""
    B, N = frame_off.shape[0] - 1, frame_entropy.shape[0]
    if frame_entropy.dtype != torch.float32 or frame_off.dtype != torch.int64:
        raise TypeError("frame_entropy must be float32 and frame_off int64")
    if out is None:
        out = alloc_gate_outputs(B, frame_entropy.device)
    rc = lib().ssd_entropy_gate(
        _dev(frame_entropy, "frame_entropy"), _dev(frame_off, "frame_off"), B, N,
        C.c_float(tau_ctc), _dev(out["gate_accept"], "gate_accept"),
        _dev(out["max_entropy"], "max_entropy"), _dev(out.get("argmax_frame"), "argmax_frame"),
        None, None, _stream())
    if rc != OK:
        raise SsdError(rc, "ssd_entropy_gate")
    return out


def _gate_from_maxima_args(utt_max_entropy, utt_status, tau_ctc, out):
    B = utt_max_entropy.shape[0]
    if utt_max_entropy.dtype != torch.float32 or utt_status.dtype != torch.int32:
        raise TypeError("utt_max_entropy must be float32 and utt_status int32 (the bits of a uint32)")
    return [None, None, B, 0, C.c_float(tau_ctc), _dev(out["gate_accept"], "gate_accept"),
            _dev(out["max_entropy"], "max_entropy"), None,
            _dev(utt_max_entropy, "utt_max_entropy"), _dev(utt_status, "utt_status"), _stream()]


def ssd_entropy_gate_from_maxima(utt_max_entropy: torch.Tensor, utt_status: torch.Tensor,
                                 tau_ctc: float, out=None) -> Dict[str, torch.Tensor]:
    """The entropy gate (Eq. 3) through ssd_entropy_gate's second form: from the utterance
    maxima and status words ssd_ctc_draft left behind (B values instead of N frame entropies).
    `out` needs gate_accept and max_entropy only."""
    if out is None:
        B, dev = utt_max_entropy.shape[0], utt_max_entropy.device
        out = dict(gate_accept=torch.empty((B,), dtype=torch.uint8, device=dev),
                   max_entropy=torch.empty((B,), dtype=torch.float32, device=dev))
    rc = lib().ssd_entropy_gate(*_gate_from_maxima_args(utt_max_entropy, utt_status, tau_ctc, out))
    if rc != OK:
        raise SsdError(rc, "ssd_entropy_gate")
    return out


def alloc_verify_outputs(M: int, B: int, device, workspace_bytes: int) -> Dict[str, torch.Tensor]:
    e = lambda n, dt: torch.empty((n,), dtype=dt, device=device)
    return dict(token_logp=e(M, torch.float32), row_lse=e(M, torch.float32),
                accepted_len=e(B, torch.int32), all_accepted=e(B, torch.uint8),
                utt_status=e(B, torch.int32),
                workspace=torch.empty((max(workspace_bytes, 256),), dtype=torch.uint8,
                                      device=device))


def ssd_verify(logits: torch.Tensor, tok_off: torch.Tensor, draft_ids: torch.Tensor,
               tau_slm: float, skip: Optional[torch.Tensor] = None, V: Optional[int] = None,
               out=None, opts: Optional[LaunchOpts] = None) -> Dict[str, torch.Tensor]:
    """Stage 2 (Eq. 5, Section 2.3): draft-token log-likelihoods and the accepted prefix."""
    M, ld = _rows_ld(logits)
    V = logits.shape[1] if V is None else V
    B = tok_off.shape[0] - 1
    if tok_off.dtype != torch.int64 or draft_ids.dtype != torch.int32:
        raise TypeError("tok_off must be int64 and draft_ids int32")
    if skip is not None and skip.dtype != torch.uint8:
        raise TypeError("skip must be uint8")
    code = _dtype_code(logits)
    if out is None:
        out = alloc_verify_outputs(M, B, logits.device,
                                   ssd_verify_workspace_bytes(B, M, V, code, opts))
    ws = out["workspace"]
    rc = lib().ssd_verify(
        _dev(logits, "logits"), code, V, ld, _dev(tok_off, "tok_off"),
        _dev(draft_ids, "draft_ids"), B, M, C.c_float(tau_slm), _dev(skip, "skip"),
        _dev(out["token_logp"], "token_logp"), _dev(out.get("row_lse"), "row_lse"),
        _dev(out["accepted_len"], "accepted_len"), _dev(out["all_accepted"], "all_accepted"),
        _dev(out["utt_status"], "utt_status"), _dev(ws, "workspace"), ws.numel(), _stream(),
        _opts(opts))
    if rc != OK:
        raise SsdError(rc, "ssd_verify")
    return out


def ssd_verify_static(logits: torch.Tensor, tok_off: torch.Tensor, draft_ids: torch.Tensor,
                      tau_slm: float, out: Dict[str, torch.Tensor],
                      skip: Optional[torch.Tensor] = None, V: Optional[int] = None,
                      opts: Optional[LaunchOpts] = None) -> Dict[str, torch.Tensor]:
    """ssd_verify for callers that cannot allocate: the scratch is the library's own fixed
    device array, so `out` holds only the result tensors (token_logp, row_lse, accepted_len,
    all_accepted, utt_status), which the caller owns and must pass in.  This wrapper allocates
    nothing either.  Sizes beyond the fixed array raise SsdError with code ERR_TOO_LARGE."""
    M, ld = _rows_ld(logits)
    V = logits.shape[1] if V is None else V
    B = tok_off.shape[0] - 1
    if tok_off.dtype != torch.int64 or draft_ids.dtype != torch.int32:
        raise TypeError("tok_off must be int64 and draft_ids int32")
    if skip is not None and skip.dtype != torch.uint8:
        raise TypeError("skip must be uint8")
    rc = lib().ssd_verify_static(
        _dev(logits, "logits"), _dtype_code(logits), V, ld, _dev(tok_off, "tok_off"),
        _dev(draft_ids, "draft_ids"), B, M, C.c_float(tau_slm), _dev(skip, "skip"),
        _dev(out["token_logp"], "token_logp"), _dev(out.get("row_lse"), "row_lse"),
        _dev(out["accepted_len"], "accepted_len"), _dev(out["all_accepted"], "all_accepted"),
        _dev(out["utt_status"], "utt_status"), _stream(), _opts(opts))
    if rc != OK:
        raise SsdError(rc, "ssd_verify_static")
    return out


def ssd_verify_shard(logits: torch.Tensor, col0: int, tok_off: torch.Tensor,
                     draft_ids: torch.Tensor, skip: Optional[torch.Tensor] = None,
                     V_local: Optional[int] = None, stats: Optional[torch.Tensor] = None,
                     workspace: Optional[torch.Tensor] = None,
                     opts: Optional[LaunchOpts] = None) -> torch.Tensor:
    """Stage 2 over a vocabulary-parallel LLM head, this rank's part: `logits` holds columns
    [col0, col0 + V_local) of the whole vocabulary; returns [M, 3] (max, sum, draft logit)."""
    M, ld = _rows_ld(logits)
    V_local = logits.shape[1] if V_local is None else V_local
    B = tok_off.shape[0] - 1
    if tok_off.dtype != torch.int64 or draft_ids.dtype != torch.int32:
        raise TypeError("tok_off must be int64 and draft_ids int32")
    if skip is not None and skip.dtype != torch.uint8:
        raise TypeError("skip must be uint8")
    if stats is None:
        stats = torch.zeros((M, 3), dtype=torch.float32, device=logits.device)
    if workspace is None:
        need = ssd_verify_workspace_bytes(B, M, V_local, _dtype_code(logits), opts)
        workspace = torch.empty((max(need, 256),), dtype=torch.uint8, device=logits.device)
    rc = lib().ssd_verify_shard(
        _dev(logits, "logits"), _dtype_code(logits), V_local, ld, col0, _dev(tok_off, "tok_off"),
        _dev(draft_ids, "draft_ids"), B, M, _dev(skip, "skip"), _dev(stats, "shard_stats"),
        _dev(workspace, "workspace"), workspace.numel(), _stream(), _opts(opts))
    if rc != OK:
        raise SsdError(rc, "ssd_verify_shard")
    return stats


def ssd_verify_combine(stats_all: torch.Tensor, V_total: int, tok_off: torch.Tensor,
                       draft_ids: torch.Tensor, tau_slm: float,
                       skip: Optional[torch.Tensor] = None, out=None) -> Dict[str, torch.Tensor]:
    """After the all-gather of every rank's ssd_verify_shard result into stats_all [R, M, 3]:
    log-likelihoods (Eq. 5) and the accepted prefix, as ssd_verify returns them."""
    if stats_all.dim() != 3 or stats_all.shape[2] != 3 or not stats_all.is_contiguous() \
            or stats_all.dtype != torch.float32:
        raise ValueError("stats_all must be a contiguous float32 tensor [R, M, 3]")
    R, M = stats_all.shape[0], stats_all.shape[1]
    B = tok_off.shape[0] - 1
    if tok_off.dtype != torch.int64 or draft_ids.dtype != torch.int32:
        raise TypeError("tok_off must be int64 and draft_ids int32")
    if out is None:
        out = alloc_verify_outputs(M, B, stats_all.device, 0)
    rc = lib().ssd_verify_combine(
        _dev(stats_all, "stats_all"), R, V_total, _dev(tok_off, "tok_off"),
        _dev(draft_ids, "draft_ids"), B, M, C.c_float(tau_slm), _dev(skip, "skip"),
        _dev(out["token_logp"], "token_logp"), _dev(out.get("row_lse"), "row_lse"),
        _dev(out["accepted_len"], "accepted_len"), _dev(out["all_accepted"], "all_accepted"),
        _dev(out["utt_status"], "utt_status"), _stream())
    if rc != OK:
        raise SsdError(rc, "ssd_verify_combine")
    return out


def ssd_verify_early_exit_workspace_bytes(B, M, V, dtype_code, opts=None) -> int:
    return int(lib().ssd_verify_early_exit_workspace_bytes(B, M, V, dtype_code, _opts(opts)))


def _early_exit_args(logits, tok_off, draft_ids, tau_slm, out, skip, V, opts):
    M, ld = _rows_ld(logits)
    V = logits.shape[1] if V is None else V
    B = tok_off.shape[0] - 1
    if tok_off.dtype != torch.int64 or draft_ids.dtype != torch.int32:
        raise TypeError("tok_off must be int64 and draft_ids int32")
    if skip is not None and skip.dtype != torch.uint8:
        raise TypeError("skip must be uint8")
    ws = out["workspace"]
    return [_dev(logits, "logits"), _dtype_code(logits), V, ld, _dev(tok_off, "tok_off"),
            _dev(draft_ids, "draft_ids"), B, M, C.c_float(tau_slm), _dev(skip, "skip"),
            _dev(out["token_logp"], "token_logp"), _dev(out.get("row_lse"), "row_lse"),
            _dev(out["accepted_len"], "accepted_len"), _dev(out["all_accepted"], "all_accepted"),
            _dev(out["utt_status"], "utt_status"), _dev(out.get("rows_read"), "rows_read"),
            _dev(ws, "workspace"), ws.numel(), _stream(), _opts(opts)]


def alloc_early_exit_outputs(M, B, V, dtype_code, device, opts=None) -> Dict[str, torch.Tensor]:
    out = alloc_verify_outputs(M, B, device,
                               ssd_verify_early_exit_workspace_bytes(B, M, V, dtype_code, opts))
    out["rows_read"] = torch.empty((B,), dtype=torch.int32, device=device)
    return out


def ssd_verify_early_exit(logits: torch.Tensor, tok_off: torch.Tensor, draft_ids: torch.Tensor,
                          tau_slm: float, skip: Optional[torch.Tensor] = None,
                          V: Optional[int] = None, out=None,
                          opts: Optional[LaunchOpts] = None) -> Dict[str, torch.Tensor]:
    """Stage 2 with early exit (Section 2.3 needs only the first reject): same decisions as
    ssd_verify; token_logp only for the rows that were read."""
    if out is None:
        M = logits.shape[0]
        out = alloc_early_exit_outputs(M, tok_off.shape[0] - 1,
                                       logits.shape[1] if V is None else V, _dtype_code(logits),
                                       logits.device, opts)
    rc = lib().ssd_verify_early_exit(*_early_exit_args(logits, tok_off, draft_ids, tau_slm, out,
                                                       skip, V, opts))
    if rc != OK:
        raise SsdError(rc, "ssd_verify_early_exit")
    return out


def bind_verify_early_exit(logits, tok_off, draft_ids, tau_slm, out, skip=None, V=None,
                           opts: Optional[LaunchOpts] = None):
    args = _early_exit_args(logits, tok_off, draft_ids, tau_slm, out, skip, V, opts)
    return BoundCall(lib().ssd_verify_early_exit, "ssd_verify_early_exit", args,
                     (logits, tok_off, draft_ids, out, skip, opts), True)


def ssd_threshold_sweep(utt_max_entropy: torch.Tensor, token_logp: torch.Tensor,
                        tok_off: torch.Tensor, tau_ctc, tau_slm, out=None,
                        want_counts: bool = True) -> Dict[str, torch.Tensor]:
    """Gate and first reject for every (tau_ctc[p], tau_slm[p]) pair from stored maxima and
    log-likelihoods (Section 3.2's operating-point sweep).  tau_ctc / tau_slm: host sequences."""
    B, M = tok_off.shape[0] - 1, token_logp.shape[0]
    P = len(tau_ctc)
    if len(tau_slm) != P:
        raise ValueError("tau_ctc and tau_slm must have the same length")
    if utt_max_entropy.dtype != torch.float32 or token_logp.dtype != torch.float32:
        raise TypeError("utt_max_entropy and token_logp must be float32")
    if tok_off.dtype != torch.int64:
        raise TypeError("tok_off must be int64")
    dev = token_logp.device if M else utt_max_entropy.device
    if out is None:
        out = dict(gate_accept=torch.empty((P, B), dtype=torch.uint8, device=dev),
                   accepted_len=torch.empty((P, B), dtype=torch.int32, device=dev),
                   all_accepted=torch.empty((P, B), dtype=torch.uint8, device=dev))
        if want_counts:
            out["counts"] = torch.empty((P, 3), dtype=torch.int32, device=dev)
    tc = (C.c_float * max(P, 1))(*[float(v) for v in tau_ctc])
    ts = (C.c_float * max(P, 1))(*[float(v) for v in tau_slm])
    rc = lib().ssd_threshold_sweep(
        _dev(utt_max_entropy, "utt_max_entropy"), _dev(token_logp, "token_logp"),
        _dev(tok_off, "tok_off"), B, M, C.cast(tc, C.c_void_p), C.cast(ts, C.c_void_p), P,
        _dev(out["gate_accept"], "gate_accept"), _dev(out["accepted_len"], "accepted_len"),
        _dev(out["all_accepted"], "all_accepted"), _dev(out.get("counts"), "counts"), _stream())
    if rc != OK:
        raise SsdError(rc, "ssd_threshold_sweep")
    return out


def ssd_assemble(tokens: torch.Tensor, tok_off: torch.Tensor, gate_accept: torch.Tensor,
                 accepted_len: torch.Tensor, all_accepted: torch.Tensor,
                 out=None) -> Dict[str, torch.Tensor]:
    """Eq. 7: final hypotheses and the ordered list of utterances left to the AR pass."""
    B, M = tok_off.shape[0] - 1, tokens.shape[0]
    if tokens.dtype != torch.int32 or accepted_len.dtype != torch.int32:
        raise TypeError("tokens and accepted_len must be int32")
    if gate_accept.dtype != torch.uint8 or all_accepted.dtype != torch.uint8:
        raise TypeError("gate_accept and all_accepted must be uint8")
    if tok_off.dtype != torch.int64:
        raise TypeError("tok_off must be int64")
    dev = tok_off.device
    if out is None:
        e = lambda n, dt: torch.empty((n,), dtype=dt, device=dev)
        out = dict(final_tokens=e(M, torch.int32), final_len=e(B, torch.int32),
                   is_final=e(B, torch.uint8), ar_count=e(1, torch.int32),
                   ar_utt=e(B, torch.int32), ar_resume=e(B, torch.int32))
    rc = lib().ssd_assemble(
        _dev(tokens, "tokens"), _dev(tok_off, "tok_off"), B, M, _dev(gate_accept, "gate_accept"),
        _dev(accepted_len, "accepted_len"), _dev(all_accepted, "all_accepted"),
        _dev(out["final_tokens"], "final_tokens"), _dev(out["final_len"], "final_len"),
        _dev(out["is_final"], "is_final"), _dev(out["ar_count"], "ar_count"),
        _dev(out["ar_utt"], "ar_utt"), _dev(out["ar_resume"], "ar_resume"), _stream())
    if rc != OK:
        raise SsdError(rc, "ssd_assemble")
    return out


def ssd_greedy_step_workspace_bytes(R, V, dtype_code, opts=None) -> int:
    return int(lib().ssd_greedy_step_workspace_bytes(R, V, dtype_code, _opts(opts)))


def ssd_greedy_step(logits: torch.Tensor, V: Optional[int] = None, out=None,
                    opts: Optional[LaunchOpts] = None) -> Dict[str, torch.Tensor]:
    """One greedy decoding step (Eq. 6) per row: most likely token and its log-likelihood."""
    R, ld = _rows_ld(logits)
    V = logits.shape[1] if V is None else V
    code = _dtype_code(logits)
    if out is None:
        dev = logits.device
        e = lambda n, dt: torch.empty((n,), dtype=dt, device=dev)
        out = dict(next_token=e(R, torch.int32), next_logp=e(R, torch.float32),
                   row_lse=e(R, torch.float32), row_status=e(R, torch.int32),
                   workspace=torch.empty((max(ssd_greedy_step_workspace_bytes(R, V, code, opts), 256),),
                                         dtype=torch.uint8, device=dev))
    ws = out["workspace"]
    rc = lib().ssd_greedy_step(
        _dev(logits, "logits"), code, V, ld, R, _dev(out["next_token"], "next_token"),
        _dev(out.get("next_logp"), "next_logp"), _dev(out.get("row_lse"), "row_lse"),
        _dev(out.get("row_status"), "row_status"), _dev(ws, "workspace"), ws.numel(), _stream(),
        _opts(opts))
    if rc != OK:
        raise SsdError(rc, "ssd_greedy_step")
    return out


class BoundCall:
    """One C-ABI call with its arguments already marshalled, for loops that issue the same call
    many times (benchmarks, serving loops): calling it enqueues the work again on the stream
    that was current when it was bound.  `opts` replaces the launch options for one call."""

    def __init__(self, fn, name: str, args: List, keep: tuple, has_opts: bool):
        self._fn, self._name, self._args, self._keep, self._has_opts = fn, name, args, keep, has_opts

    def __call__(self, opts: Optional[LaunchOpts] = None) -> None:
        a = self._args
        if opts is not None:
            if not self._has_opts:
                raise TypeError(self._name + " takes no launch options")
            a = a[:-1] + [C.cast(C.pointer(opts), C.c_void_p)]
        rc = self._fn(*a)
        if rc != OK:
            raise SsdError(rc, self._name)


def bind_ctc_draft(logits, frame_off, blank_id, max_draft_len, out, V=None,
                   opts: Optional[LaunchOpts] = None) -> BoundCall:
    N, ld = _rows_ld(logits)
    V = logits.shape[1] if V is None else V
    B = frame_off.shape[0] - 1
    args = [_dev(logits, "logits"), _dtype_code(logits), V, ld, _dev(frame_off, "frame_off"), B, N,
            blank_id, max_draft_len, _dev(out["frame_entropy"], "frame_entropy"),
            _dev(out["frame_argmax"], "frame_argmax"), _dev(out.get("frame_lse"), "frame_lse"),
            None, _dev(out["draft_tokens"], "draft_tokens"),
            _dev(out.get("draft_frames"), "draft_frames"), _dev(out["draft_len"], "draft_len"),
            _dev(out["draft_full_len"], "draft_full_len"),
            _dev(out["utt_max_entropy"], "utt_max_entropy"), _dev(out["utt_status"], "utt_status"),
            _dev(out.get("workspace"), "workspace"),
            0 if out.get("workspace") is None else out["workspace"].numel(), _stream(), _opts(opts)]
    return BoundCall(lib().ssd_ctc_draft, "ssd_ctc_draft", args, (logits, frame_off, out, opts), True)


def bind_entropy_gate(frame_entropy, frame_off, tau_ctc, out) -> BoundCall:
    B, N = frame_off.shape[0] - 1, frame_entropy.shape[0]
    args = [_dev(frame_entropy, "frame_entropy"), _dev(frame_off, "frame_off"), B, N,
            C.c_float(tau_ctc), _dev(out["gate_accept"], "gate_accept"),
            _dev(out["max_entropy"], "max_entropy"), _dev(out.get("argmax_frame"), "argmax_frame"),
            None, None, _stream()]
    return BoundCall(lib().ssd_entropy_gate, "ssd_entropy_gate", args,
                     (frame_entropy, frame_off, out), False)


def bind_entropy_gate_from_maxima(utt_max_entropy, utt_status, tau_ctc, out) -> BoundCall:
    return BoundCall(lib().ssd_entropy_gate, "ssd_entropy_gate",
                     _gate_from_maxima_args(utt_max_entropy, utt_status, tau_ctc, out),
                     (utt_max_entropy, utt_status, out), False)


def bind_verify(logits, tok_off, draft_ids, tau_slm, out, skip=None, V=None,
                opts: Optional[LaunchOpts] = None) -> BoundCall:
    M, ld = _rows_ld(logits)
    V = logits.shape[1] if V is None else V
    B = tok_off.shape[0] - 1
    ws = out["workspace"]
    args = [_dev(logits, "logits"), _dtype_code(logits), V, ld, _dev(tok_off, "tok_off"),
            _dev(draft_ids, "draft_ids"), B, M, C.c_float(tau_slm), _dev(skip, "skip"),
            _dev(out["token_logp"], "token_logp"), _dev(out.get("row_lse"), "row_lse"),
            _dev(out["accepted_len"], "accepted_len"), _dev(out["all_accepted"], "all_accepted"),
            _dev(out["utt_status"], "utt_status"), _dev(ws, "workspace"), ws.numel(), _stream(),
            _opts(opts)]
    return BoundCall(lib().ssd_verify, "ssd_verify", args,
                     (logits, tok_off, draft_ids, out, skip, opts), True)
