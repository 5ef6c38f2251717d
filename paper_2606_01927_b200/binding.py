"""ctypes binding of ``libalbireo_sample.so`` -- argument marshalling only.

Every step of the sampling path runs inside the CUDA library; this module only turns
torch tensors (device memory, streams) into the pointers and sizes of the C ABI declared
in ``include/albireo_sample.h``.  There is no CPU fallback: if the library is missing or
does not load, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

from . import _build

F32 = 0
BF16 = 1
F16 = 2


def _dtype_code(t: torch.Tensor) -> int:
    try:
        return {torch.float32: F32, torch.bfloat16: BF16, torch.float16: F16}[t.dtype]
    except KeyError:
        raise ValueError("logits must be float32, bfloat16 or float16") from None
OK, EINVAL, ENOMEM, ECUDA, EUNSUPPORTED = 0, -1, -2, -3, -4
ROW_GENERAL_PATH, ROW_BAD_PARAM, ROW_HISTORY_OVERFLOW, ROW_TIMEOUT = 1, 2, 4, 8
FLAG_FORCE_GENERAL = 1
FLAG_TOPK_KEEP_TIES = 2
FLAG_LOGPROB_FULL_VOCAB = 4
FLAG_PROGRAMMATIC_LAUNCH = 8
MAX_VOCAB = 524288
MAX_NUM_TOP = 128
FIXED_MAX_HISTORY = 1 << 20

EXPORTS = [
    "albireo_sample_workspace_bytes", "albireo_sample_host_staging_bytes", "albireo_sample_init",
    "albireo_sample", "albireo_sample_host", "albireo_sample_destroy", "albireo_last_error",
    "albireo_sample_launch_count", "albireo_sample_fixed_scratch", "albireo_sample_fixed_scratch_error",
    "albireo_stream_only",
]


class SampleExt(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("flags", C.c_uint32), ("row_stride_elems", C.c_int64),
        ("row_base", C.c_uint32), ("num_top", C.c_int32),
        ("out_top_ids", C.c_void_p), ("out_top_logprobs", C.c_void_p),
        ("out_num_kept", C.c_void_p), ("out_num_topk", C.c_void_p),
        ("dbg_cap", C.c_int32), ("dbg_topk_ids", C.c_void_p), ("out_row_status", C.c_void_p),
        ("exp1", C.c_void_p), ("exp1_stride_elems", C.c_int64),
        ("backfill_ids", C.c_void_p), ("backfill_index", C.c_void_p), ("backfill_len", C.c_int64),
        ("feedback_ring", C.c_void_p), ("feedback_cap", C.c_int64), ("feedback_head", C.c_int64),
        ("num_segments", C.c_int32), ("segment_stride_elems", C.c_int64),
        ("history_output_start", C.c_void_p),
        ("segment_ptrs", C.c_void_p), ("segment_row_offset", C.c_int64),
    ]


def _load() -> C.CDLL:
    path = _build.LIB_PATH
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -c 'import __graft_entry__ as g; g.build()'` "
            "(nvcc, sm_100a). The sampler has no CPU fallback.")
    lib = C.CDLL(path)
    for name in EXPORTS:
        if not hasattr(lib, name):
            raise ImportError(f"{path} does not export {name}")
    vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
    lib.albireo_sample_workspace_bytes.restype = C.c_size_t
    lib.albireo_sample_workspace_bytes.argtypes = [i32, i32, i64]
    lib.albireo_sample_host_staging_bytes.restype = C.c_size_t
    lib.albireo_sample_host_staging_bytes.argtypes = [i32, i32, i64]
    lib.albireo_sample_init.restype = C.c_int
    lib.albireo_sample_init.argtypes = [C.POINTER(vp), i32, i32, i32, i64, vp, C.c_size_t]
    sample_args = [vp, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, u64, vp, vp, vp, C.POINTER(SampleExt)]
    lib.albireo_sample.restype = C.c_int
    lib.albireo_sample.argtypes = sample_args
    lib.albireo_sample_host.restype = C.c_int
    lib.albireo_sample_host.argtypes = sample_args[:14] + [i64] + sample_args[14:]
    lib.albireo_sample_destroy.restype = C.c_int
    lib.albireo_sample_destroy.argtypes = [vp]
    lib.albireo_last_error.restype = C.c_char_p
    lib.albireo_last_error.argtypes = [vp]
    lib.albireo_sample_launch_count.restype = C.c_uint64
    lib.albireo_sample_launch_count.argtypes = [vp]
    lib.albireo_sample_fixed_scratch.restype = C.c_int
    lib.albireo_sample_fixed_scratch.argtypes = sample_args[1:14] + [i64] + sample_args[14:]
    lib.albireo_sample_fixed_scratch_error.restype = C.c_char_p
    lib.albireo_sample_fixed_scratch_error.argtypes = []
    lib.albireo_stream_only.restype = C.c_int
    lib.albireo_stream_only.argtypes = [vp, vp, i32, i32, i32, vp, i32, vp]
    return lib


LIB = _load()


class AlbireoError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"albireo_sample error {code}: {msg}")
        self.code = code


def albireo_sample_workspace_bytes(max_rows: int, max_vocab: int, max_history_total: int) -> int:
    return int(LIB.albireo_sample_workspace_bytes(max_rows, max_vocab, max_history_total))


def albireo_sample_host_staging_bytes(max_rows: int, max_vocab: int, max_history_total: int) -> int:
    return int(LIB.albireo_sample_host_staging_bytes(max_rows, max_vocab, max_history_total))


def _dp(t: Optional[torch.Tensor], dtype, device_type: str):
    if t is None:
        return None
    if t.dtype != dtype or not t.is_contiguous() or t.device.type != device_type:
        raise ValueError(f"expected contiguous {dtype} tensor on {device_type}, got {t.dtype} on {t.device}")
    return C.c_void_p(t.data_ptr())


@dataclass
class SampleOutputs:
    tokens: torch.Tensor
    logprobs: torch.Tensor
    top_ids: Optional[torch.Tensor] = None
    top_logprobs: Optional[torch.Tensor] = None
    num_kept: Optional[torch.Tensor] = None
    num_topk: Optional[torch.Tensor] = None
    dbg_topk_ids: Optional[torch.Tensor] = None
    row_status: Optional[torch.Tensor] = None


class Sampler:
    """Owns a handle from ``albireo_sample_init`` and the torch-allocated workspace."""

    def __init__(self, max_rows: int, max_vocab: int, max_history_total: int = 0,
                 device: Optional[torch.device] = None, host_staging: bool = False):
        if not torch.cuda.is_available():
            raise RuntimeError("albireo sampler needs a CUDA device; there is no CPU path")
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        self.max_rows, self.max_vocab, self.max_history_total = max_rows, max_vocab, max_history_total
        nbytes = albireo_sample_workspace_bytes(max_rows, max_vocab, max_history_total)
        if host_staging:
            nbytes += albireo_sample_host_staging_bytes(max_rows, max_vocab, max_history_total)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = self.workspace.data_ptr()
        self._ws_ptr = (base + 255) & ~255
        self._handle = C.c_void_p()
        with torch.cuda.device(self.device):
            rc = LIB.albireo_sample_init(C.byref(self._handle), self.device.index, max_rows, max_vocab,
                                         max_history_total, C.c_void_p(self._ws_ptr), nbytes)
        if rc != OK:
            raise AlbireoError(rc, "albireo_sample_init failed")

    # -- raw pass-through ------------------------------------------------------------
    def last_error(self) -> str:
        return LIB.albireo_last_error(self._handle).decode()

    def launch_count(self) -> int:
        return int(LIB.albireo_sample_launch_count(self._handle))

    def close(self):
        if getattr(self, "_handle", None) is not None and self._handle:
            LIB.albireo_sample_destroy(self._handle)
            self._handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _ext(self, B, dev_type, device, *, row_base=0, row_stride=0, num_top=0, want_counts=False,
             dbg_cap=0, want_status=False, flags=0, out_top_ids=None, out_top_logprobs=None):
        ext = SampleExt()
        ext.struct_size = C.sizeof(SampleExt)
        ext.flags = flags
        ext.row_stride_elems = row_stride
        ext.row_base = row_base
        ext.num_top = num_top
        out = {}
        kw = dict(device=device) if dev_type == "cuda" else dict(pin_memory=True)
        if num_top > 0:
            if out_top_ids is not None and (out_top_ids.dtype != torch.int32 or out_top_ids.numel() < B * num_top
                                            or not out_top_ids.is_contiguous()):
                raise ValueError("out_top_ids must be a contiguous int32 tensor of B * num_top entries")
            if out_top_logprobs is not None and (out_top_logprobs.dtype != torch.float32 or out_top_logprobs.numel() < B * num_top
                                                 or not out_top_logprobs.is_contiguous()):
                raise ValueError("out_top_logprobs must be a contiguous float32 tensor of B * num_top entries")
            out["top_ids"] = torch.empty((B, num_top), dtype=torch.int32, **kw) if out_top_ids is None else out_top_ids
            out["top_logprobs"] = (torch.empty((B, num_top), dtype=torch.float32, **kw)
                                   if out_top_logprobs is None else out_top_logprobs)
            ext.out_top_ids = out["top_ids"].data_ptr()
            ext.out_top_logprobs = out["top_logprobs"].data_ptr()
        if want_counts:
            out["num_kept"] = torch.empty(B, dtype=torch.int32, **kw)
            out["num_topk"] = torch.empty(B, dtype=torch.int32, **kw)
            ext.out_num_kept = out["num_kept"].data_ptr()
            ext.out_num_topk = out["num_topk"].data_ptr()
        if dbg_cap > 0:
            out["dbg_topk_ids"] = torch.empty((B, dbg_cap), dtype=torch.int32, **kw)
            ext.dbg_cap = dbg_cap
            ext.dbg_topk_ids = out["dbg_topk_ids"].data_ptr()
        if want_status:
            out["row_status"] = torch.empty(B, dtype=torch.int32, **kw)
            ext.out_row_status = out["row_status"].data_ptr()
        return ext, out

    def albireo_sample(self, logits: torch.Tensor, *, temperature=None, top_k=None, top_p=None, min_p=None,
                       repetition_penalty=None, presence_penalty=None, frequency_penalty=None,
                       history_ids=None, history_offsets=None, seeds=None, step: int = 0,
                       out_tokens=None, out_logprobs=None, stream: Optional[torch.cuda.Stream] = None,
                       row_base: int = 0, num_top: int = 0, want_counts=False, dbg_cap: int = 0,
                       want_status=False, flags: int = 0, B: Optional[int] = None, V: Optional[int] = None,
                       exp1: Optional[torch.Tensor] = None, backfill_ids: Optional[torch.Tensor] = None,
                       backfill_index: Optional[torch.Tensor] = None, feedback_ring: Optional[torch.Tensor] = None,
                       feedback_head: int = 0, output_start: Optional[torch.Tensor] = None,
                       segment_tensors=None, segment_row_offset: int = 0,
                       out_top_ids: Optional[torch.Tensor] = None,
                       out_top_logprobs: Optional[torch.Tensor] = None) -> SampleOutputs:
        """Device-resident call: all tensors on ``self.device``; asynchronous on ``stream``.

        ``exp1`` (float32 ``[B, V]``) replaces the counter-based draw by pre-generated Exp(1)
        variates; ``backfill_ids`` / ``backfill_index`` (int32) and ``feedback_ring`` (int64,
        device or pinned host memory) are the early-feedback targets."""
        nseg = 0
        if logits.dim() == 3:
            # rows in pieces, [t, B, V / t]: the receive buffer of the sequence-parallel all-to-all
            if logits.stride(2) != 1:
                raise ValueError("logits in pieces must be [t, B, V/t] with unit stride along the last axis")
            nseg = logits.shape[0]
            B = logits.shape[1] if B is None else B
            V = nseg * logits.shape[2] if V is None else V
        elif logits.dim() != 2 or logits.stride(1) != 1:
            raise ValueError("logits must be [B, V] with unit stride along V")
        else:
            B = logits.shape[0] if B is None else B
            V = logits.shape[1] if V is None else V
        dt = _dtype_code(logits)
        dev = logits.device
        if out_tokens is None:
            out_tokens = torch.empty(B, dtype=torch.int32, device=dev)
        if out_logprobs is None:
            out_logprobs = torch.empty(B, dtype=torch.float32, device=dev)
        row_stride = logits.stride(0) if B > 1 else V
        if nseg:
            row_stride = logits.stride(1)
        ext, extra = self._ext(B, "cuda", dev, row_base=row_base, row_stride=0 if row_stride == V else row_stride,
                               num_top=num_top, want_counts=want_counts, dbg_cap=dbg_cap,
                               want_status=want_status, flags=flags, out_top_ids=out_top_ids,
                               out_top_logprobs=out_top_logprobs)
        if nseg:
            ext.num_segments = nseg
            ext.segment_stride_elems = logits.stride(0)
            ext.row_stride_elems = row_stride
        if output_start is not None:
            ext.history_output_start = _dp(output_start, torch.int32, "cuda")
        if segment_tensors is not None:
            # one [rows, V/t] buffer per piece (e.g. the peers' vocabulary shards in symmetric memory), read in place
            t_ = len(segment_tensors)
            sh0 = segment_tensors[0]
            if any(x.dim() != 2 or x.stride(1) != 1 or x.dtype != sh0.dtype or x.shape[1] != sh0.shape[1]
                   or x.stride(0) != sh0.stride(0) for x in segment_tensors):
                raise ValueError("segment_tensors must be same-shaped [rows, V/t] tensors with unit stride along V/t")
            ptrs = (C.c_void_p * t_)(*[x.data_ptr() for x in segment_tensors])
            ext.num_segments = t_
            ext.segment_ptrs = C.cast(ptrs, C.c_void_p)
            ext.segment_row_offset = segment_row_offset
            ext.row_stride_elems = sh0.stride(0)
            ext._keepalive = ptrs
        if exp1 is not None:
            if exp1.dtype != torch.float32 or exp1.dim() != 2 or exp1.stride(1) != 1 or exp1.device != dev:
                raise ValueError("exp1 must be a float32 [B, V] tensor on the logits' device")
            ext.exp1 = exp1.data_ptr()
            ext.exp1_stride_elems = 0 if (B <= 1 or exp1.stride(0) == V) else exp1.stride(0)
        if backfill_ids is not None:
            ext.backfill_ids = _dp(backfill_ids, torch.int32, "cuda")
            ext.backfill_index = _dp(backfill_index, torch.int32, "cuda")
            ext.backfill_len = backfill_ids.numel()
        if feedback_ring is not None:
            if feedback_ring.dtype != torch.int64 or not feedback_ring.is_contiguous():
                raise ValueError("feedback_ring must be a contiguous int64 tensor (device, or pinned host memory)")
            ext.feedback_ring = feedback_ring.data_ptr()
            ext.feedback_cap = feedback_ring.numel()
            ext.feedback_head = feedback_head
        st = torch.cuda.current_stream(dev) if stream is None else stream
        f32, i32 = torch.float32, torch.int32
        with torch.cuda.device(dev):
            rc = LIB.albireo_sample(
                self._handle, C.c_void_p(logits.data_ptr()), B, V, dt,
                _dp(temperature, f32, "cuda"), _dp(top_k, i32, "cuda"), _dp(top_p, f32, "cuda"), _dp(min_p, f32, "cuda"),
                _dp(repetition_penalty, f32, "cuda"), _dp(presence_penalty, f32, "cuda"),
                _dp(frequency_penalty, f32, "cuda"), _dp(history_ids, i32, "cuda"), _dp(history_offsets, i32, "cuda"),
                _dp(seeds, torch.int64, "cuda"), C.c_uint64(step),
                C.c_void_p(out_tokens.data_ptr()), C.c_void_p(out_logprobs.data_ptr()),
                C.c_void_p(st.cuda_stream), C.byref(ext))
        if rc != OK:
            raise AlbireoError(rc, self.last_error())
        return SampleOutputs(out_tokens, out_logprobs, **extra)

    def albireo_stream_only(self, logits: torch.Tensor, sink: torch.Tensor, stream: Optional[torch.cuda.Stream] = None,
                            drop_tile: int = -1):
        """Measurement aid: the sampler's stream over ``logits`` ([B, V], dense) and nothing else.
        ``drop_tile >= 0`` withholds that tile's copy so that the bounded wait on it expires (bit 31 of the sink words)."""
        B, V = logits.shape
        if not logits.is_contiguous() or sink.dtype != torch.int32 or sink.numel() < B:
            raise ValueError("albireo_stream_only wants dense logits and an int32 sink of B words")
        st = torch.cuda.current_stream(logits.device) if stream is None else stream
        with torch.cuda.device(logits.device):
            rc = LIB.albireo_stream_only(self._handle, C.c_void_p(logits.data_ptr()), B, V, _dtype_code(logits),
                                         C.c_void_p(sink.data_ptr()), int(drop_tile), C.c_void_p(st.cuda_stream))
        if rc != OK:
            raise AlbireoError(rc, self.last_error())

    def albireo_sample_host(self, logits: torch.Tensor, *, temperature=None, top_k=None, top_p=None, min_p=None,
                            repetition_penalty=None, presence_penalty=None, frequency_penalty=None,
                            history_ids=None, history_offsets=None, seeds=None, step: int = 0,
                            out_tokens=None, out_logprobs=None, stream: Optional[torch.cuda.Stream] = None,
                            row_base: int = 0, num_top: int = 0, want_counts=False, want_status=False,
                            flags: int = 0) -> SampleOutputs:
        """Host-buffer call (CPU tensors, ideally pinned): copies in, samples, copies out, waits."""
        B, V = logits.shape
        dt = _dtype_code(logits)
        if out_tokens is None:
            out_tokens = torch.empty(B, dtype=torch.int32, pin_memory=True)
        if out_logprobs is None:
            out_logprobs = torch.empty(B, dtype=torch.float32, pin_memory=True)
        ext, extra = self._ext(B, "cpu", None, row_base=row_base, num_top=num_top, want_counts=want_counts,
                               want_status=want_status, flags=flags)
        st = torch.cuda.current_stream(self.device) if stream is None else stream
        f32, i32 = torch.float32, torch.int32
        htot = int(history_ids.numel()) if history_ids is not None else 0
        with torch.cuda.device(self.device):
            rc = LIB.albireo_sample_host(
                self._handle, C.c_void_p(logits.data_ptr()), B, V, dt,
                _dp(temperature, f32, "cpu"), _dp(top_k, i32, "cpu"), _dp(top_p, f32, "cpu"), _dp(min_p, f32, "cpu"),
                _dp(repetition_penalty, f32, "cpu"), _dp(presence_penalty, f32, "cpu"),
                _dp(frequency_penalty, f32, "cpu"), _dp(history_ids, i32, "cpu"), _dp(history_offsets, i32, "cpu"),
                C.c_int64(htot), _dp(seeds, torch.int64, "cpu"), C.c_uint64(step),
                C.c_void_p(out_tokens.data_ptr()), C.c_void_p(out_logprobs.data_ptr()),
                C.c_void_p(st.cuda_stream), C.byref(ext))
        if rc != OK:
            raise AlbireoError(rc, self.last_error())
        return SampleOutputs(out_tokens, out_logprobs, **extra)


def albireo_sample_fixed_scratch(logits: torch.Tensor, *, temperature=None, top_k=None, top_p=None, min_p=None,
                                 repetition_penalty=None, presence_penalty=None, frequency_penalty=None,
                                 history_ids=None, history_offsets=None, history_total: Optional[int] = None,
                                 seeds=None, step: int = 0, out_tokens=None, out_logprobs=None,
                                 stream: Optional[torch.cuda.Stream] = None, row_base: int = 0,
                                 want_status: bool = False, want_counts: bool = False) -> SampleOutputs:
    """The sampler for callers that may not allocate: no handle, no workspace (the library's own
    fixed scratch array is used).  The output tensors created here when none are passed (and the
    per-row status / count arrays when asked for) are a convenience of this Python wrapper; the C
    entry point itself allocates nothing."""
    B, V = logits.shape
    dt = _dtype_code(logits)
    dev = logits.device
    if out_tokens is None:
        out_tokens = torch.empty(B, dtype=torch.int32, device=dev)
    if out_logprobs is None:
        out_logprobs = torch.empty(B, dtype=torch.float32, device=dev)
    ext = SampleExt()
    ext.struct_size = C.sizeof(SampleExt)
    ext.row_base = row_base
    row_status = num_kept = num_topk = None
    if want_status:
        row_status = torch.zeros(B, dtype=torch.int32, device=dev)
        ext.out_row_status = row_status.data_ptr()
    if want_counts:
        num_kept = torch.empty(B, dtype=torch.int32, device=dev)
        num_topk = torch.empty(B, dtype=torch.int32, device=dev)
        ext.out_num_kept, ext.out_num_topk = num_kept.data_ptr(), num_topk.data_ptr()
    if history_total is None:
        history_total = int(history_ids.numel()) if history_ids is not None else 0
    st = torch.cuda.current_stream(dev) if stream is None else stream
    f32, i32 = torch.float32, torch.int32
    with torch.cuda.device(dev):
        rc = LIB.albireo_sample_fixed_scratch(
            C.c_void_p(logits.data_ptr()), B, V, dt,
            _dp(temperature, f32, "cuda"), _dp(top_k, i32, "cuda"), _dp(top_p, f32, "cuda"), _dp(min_p, f32, "cuda"),
            _dp(repetition_penalty, f32, "cuda"), _dp(presence_penalty, f32, "cuda"),
            _dp(frequency_penalty, f32, "cuda"), _dp(history_ids, i32, "cuda"), _dp(history_offsets, i32, "cuda"),
            C.c_int64(history_total), _dp(seeds, torch.int64, "cuda"), C.c_uint64(step),
            C.c_void_p(out_tokens.data_ptr()), C.c_void_p(out_logprobs.data_ptr()),
            C.c_void_p(st.cuda_stream), C.byref(ext))
    if rc != OK:
        raise AlbireoError(rc, LIB.albireo_sample_fixed_scratch_error().decode())
    return SampleOutputs(out_tokens, out_logprobs, num_kept=num_kept, num_topk=num_topk, row_status=row_status)


# ------------------------------------------------------------------ workload marshalling

def workload_tensors(w, device, pinned: bool = False) -> dict:
    """Moves a ``workloads.Workload`` (numpy) into torch tensors on ``device`` ('cpu' keeps
    them on the host, pinned if asked).  Pure data movement; seeds travel as the int64
    view of their uint64 bit patterns."""
    import numpy as np

    def conv(a, view=None):
        if a is None:
            return None
        t = torch.from_numpy(np.ascontiguousarray(a))
        if view is not None:
            t = t.view(view)
        if str(device) == "cpu":
            return t.pin_memory() if pinned else t
        return t.to(device)

    hid = w.history_ids
    if hid is not None and hid.size == 0:
        hid = np.zeros(1, dtype=np.int32)      # an empty CSR still needs a non-NULL pointer
    if w.dtype == F32:
        logits = conv(w.logits)
    elif w.dtype == F16:
        logits = conv(w.logits.view(np.int16), torch.float16)
    else:
        logits = conv(w.logits.view(np.int16), torch.bfloat16)
    extra = {}
    if getattr(w, "exp1", None) is not None:
        extra["exp1"] = conv(w.exp1)
    if getattr(w, "backfill_index", None) is not None:
        extra["backfill_index"] = conv(w.backfill_index)
    if getattr(w, "output_start", None) is not None:
        extra["output_start"] = conv(w.output_start)
    return dict(
        **extra,
        logits=logits, temperature=conv(w.temperature), top_k=conv(w.top_k), top_p=conv(w.top_p),
        min_p=conv(w.min_p), repetition_penalty=conv(w.repetition_penalty),
        presence_penalty=conv(w.presence_penalty), frequency_penalty=conv(w.frequency_penalty),
        history_ids=conv(hid), history_offsets=conv(w.history_offsets),
        seeds=conv(None if w.seeds is None else w.seeds.view(np.int64)), step=int(w.step))
