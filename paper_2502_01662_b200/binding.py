"""ctypes binding of include/cos_verify.h: argument marshalling only.

torch supplies device memory and the stream; all arithmetic happens in the CUDA library.
Loading fails loudly if the library cannot be built or opened.
"""
from __future__ import annotations

import ctypes
from typing import Optional, Sequence

from . import build as _build

COS_MAX_MODELS = 8
COS_OK = 0
COS_COMBINE_PROB_ENSEMBLE = 0
COS_COMBINE_LOGIT_LINEAR = 1
COS_DTYPE_F32 = 0
COS_DTYPE_BF16 = 1
COS_DTYPE_F16 = 2
COS_ROW_NONFINITE = 1
COS_ROW_BAD_DRAFT = 2
COS_ROW_Q_ZERO = 4
COS_ROW_RESIDUAL_EMPTY = 8
COS_ROW_FAULT = 16   # an internal wait of the kernel gave up: the call's outputs are undefined
COS_RUN_ALL_RESIDUALS = 1
COS_RUN_PROPOSER_PER_POSITION = 2   # proposer is [B, gamma+1]: the model that proposed each draft (Algorithm 2)
COS_RUN_BONUS_FROM_MODEL = 4        # the bonus token follows one named model's own distribution (Sec. 3.3)
COS_RUN_EARLY_EXIT = 8              # hint: positions behind a reported rejection may be left unread
COS_RUN_INPUTS_SETTLED = 16         # promise: the inputs were complete before the work ahead of the call in its stream was submitted

_STATUS_NAMES = {1: "COS_ERR_INVALID_ARG", 2: "COS_ERR_UNSUPPORTED", 3: "COS_ERR_ALIGNMENT",
                 4: "COS_ERR_CUDA", 5: "COS_ERR_NOMEM"}

EXPORTS = ("cos_verify_create", "cos_verify_run", "cos_verify_run_host", "cos_verify_get_info",
           "cos_verify_destroy", "cos_verify_last_error", "cos_verify_set_stage_timing", "cos_verify_get_stage_ms",
           "cos_verify_run_static", "cos_verify_set_wait_limit", "cos_verify_measure_ceiling", "cos_verify_set_one_launch")


class CosVerifyError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{_STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class cos_verify_config(ctypes.Structure):
    _fields_ = [
        ("n", ctypes.c_int32), ("combine", ctypes.c_int32), ("weights", ctypes.c_float * COS_MAX_MODELS),
        ("mask_model", ctypes.c_int32), ("mask_alpha", ctypes.c_float), ("temperature", ctypes.c_float),
        ("gamma", ctypes.c_int32), ("vocab", ctypes.c_int32), ("max_batch", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("device", ctypes.c_int32), ("cluster_size", ctypes.c_int32),
        ("host_staging", ctypes.c_int32),
    ]


class cos_verify_args(ctypes.Structure):
    _fields_ = [
        ("logits", ctypes.c_void_p), ("stride_model", ctypes.c_int64), ("stride_row", ctypes.c_int64),
        ("stride_pos", ctypes.c_int64), ("draft_tokens", ctypes.c_void_p), ("proposer", ctypes.c_void_p),
        ("batch", ctypes.c_int32), ("flags", ctypes.c_int32), ("row_base", ctypes.c_int64),
        ("seed", ctypes.c_uint64), ("offset", ctypes.c_uint64), ("accept_count", ctypes.c_void_p),
        ("out_tokens", ctypes.c_void_p), ("row_status", ctypes.c_void_p), ("diag", ctypes.c_void_p),
        ("dump_r", ctypes.c_void_p), ("bonus_prob", ctypes.c_void_p), ("bonus_model", ctypes.c_int32),
        ("offset_device", ctypes.c_void_p), ("lse", ctypes.c_void_p),
    ]


class cos_verify_info(ctypes.Structure):
    _fields_ = [
        ("cluster_size", ctypes.c_int32), ("threads_per_block", ctypes.c_int32), ("max_clusters", ctypes.c_int32),
        ("sm_count", ctypes.c_int32), ("launches_per_run", ctypes.c_int32), ("reserved", ctypes.c_int32 * 3),
    ]


_lib = None


def load_library(rebuild: bool = False) -> ctypes.CDLL:
    """Build (if stale) and open libcos_verify.so; raises if either step fails."""
    global _lib
    if _lib is not None and not rebuild:
        return _lib
    path = _build.build(force=rebuild)
    lib = ctypes.CDLL(path)
    lib.cos_verify_create.argtypes = [ctypes.POINTER(cos_verify_config), ctypes.POINTER(ctypes.c_void_p)]
    lib.cos_verify_create.restype = ctypes.c_int
    lib.cos_verify_run.argtypes = [ctypes.c_void_p, ctypes.POINTER(cos_verify_args), ctypes.c_void_p]
    lib.cos_verify_run.restype = ctypes.c_int
    lib.cos_verify_run_host.argtypes = [ctypes.c_void_p, ctypes.POINTER(cos_verify_args), ctypes.c_void_p]
    lib.cos_verify_run_host.restype = ctypes.c_int
    lib.cos_verify_get_info.argtypes = [ctypes.c_void_p, ctypes.POINTER(cos_verify_info)]
    lib.cos_verify_get_info.restype = ctypes.c_int
    lib.cos_verify_set_stage_timing.argtypes = [ctypes.c_void_p, ctypes.c_int]
    lib.cos_verify_set_stage_timing.restype = ctypes.c_int
    lib.cos_verify_get_stage_ms.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32)]
    lib.cos_verify_get_stage_ms.restype = ctypes.c_int
    lib.cos_verify_set_one_launch.argtypes = [ctypes.c_void_p, ctypes.c_int32]
    lib.cos_verify_set_one_launch.restype = ctypes.c_int
    lib.cos_verify_set_wait_limit.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_int32]
    lib.cos_verify_set_wait_limit.restype = ctypes.c_int
    lib.cos_verify_measure_ceiling.argtypes = [ctypes.c_int32, ctypes.c_void_p, ctypes.c_uint64, ctypes.c_void_p,
                                               ctypes.c_uint64, ctypes.c_int32, ctypes.POINTER(ctypes.c_float),
                                               ctypes.c_void_p]
    lib.cos_verify_measure_ceiling.restype = ctypes.c_int
    lib.cos_verify_destroy.argtypes = [ctypes.c_void_p]
    lib.cos_verify_destroy.restype = ctypes.c_int
    lib.cos_verify_last_error.argtypes = [ctypes.c_void_p]
    lib.cos_verify_last_error.restype = ctypes.c_char_p
    _lib = lib
    return lib


def _dtype_code(torch_dtype) -> int:
    import torch
    if torch_dtype == torch.float32:
        return COS_DTYPE_F32
    if torch_dtype == torch.bfloat16:
        return COS_DTYPE_BF16
    if torch_dtype == torch.float16:
        return COS_DTYPE_F16
    raise ValueError(f"logits must be float32, bfloat16 or float16, not {torch_dtype}")


class CosVerifier:
    """One verification context (cos_verify_create ... cos_verify_destroy).

    run() takes device tensors and returns device tensors; run_host() takes host tensors
    (pinned for asynchronous copies) and returns host tensors, the copies being part of the call.
    """

    def __init__(self, n: int, combine: int, weights: Sequence[float], temperature: float, gamma: int,
                 vocab: int, max_batch: int, dtype, mask_model: int = -1, mask_alpha: float = 1.0,
                 device: int = 0, cluster_size: int = 0, host_staging: bool = False):
        self._lib = load_library()
        self._ctx = ctypes.c_void_p()
        cfg = cos_verify_config()
        cfg.n, cfg.combine = n, combine
        for i, w in enumerate(list(weights)[:COS_MAX_MODELS]):
            cfg.weights[i] = w
        cfg.mask_model, cfg.mask_alpha, cfg.temperature = mask_model, mask_alpha, temperature
        cfg.gamma, cfg.vocab, cfg.max_batch = gamma, vocab, max_batch
        cfg.dtype = dtype if isinstance(dtype, int) else _dtype_code(dtype)
        cfg.device, cfg.cluster_size, cfg.host_staging = device, cluster_size, int(host_staging)
        self.cfg = cfg
        st = self._lib.cos_verify_create(ctypes.byref(cfg), ctypes.byref(self._ctx))
        if st != COS_OK:
            msg = self._lib.cos_verify_last_error(None).decode()
            self._ctx = ctypes.c_void_p()
            raise CosVerifyError(st, msg)

    # -- helpers ---------------------------------------------------------------------
    def _check(self, st: int):
        if st != COS_OK:
            raise CosVerifyError(st, self._lib.cos_verify_last_error(self._ctx).decode())

    def info(self) -> dict:
        inf = cos_verify_info()
        self._check(self._lib.cos_verify_get_info(self._ctx, ctypes.byref(inf)))
        out = {k: getattr(inf, k) for k in ("cluster_size", "threads_per_block", "max_clusters", "sm_count",
                                            "launches_per_run")}
        out["items_per_position"], out["draw_items_per_position"] = inf.reserved[0], inf.reserved[1]
        out["one_launch"] = bool(inf.reserved[2] & 1)
        out["draw_items"] = bool(inf.reserved[2] & 2)   # tokens are drawn by the persistent kernel's drawing items
        return out

    def _fill_args(self, logits, drafts, proposer, seed, offset, row_base, flags, outs,
                   bonus_model=None, offset_device=None) -> cos_verify_args:
        n, B, P, V = logits.shape
        # a [B, gamma+1] proposer table selects the per-position form; a bonus model selects its flag
        if proposer.dim() == 2:
            if tuple(proposer.shape) != (B, P):
                raise ValueError("a per-position proposer table must be [B, gamma+1]")
            flags |= COS_RUN_PROPOSER_PER_POSITION
        elif proposer.numel() != B:
            raise ValueError("proposer must be [B] or [B, gamma+1]")
        if bonus_model is not None and bonus_model >= 0:
            flags |= COS_RUN_BONUS_FROM_MODEL
        if n != self.cfg.n or P != self.cfg.gamma + 1 or V != self.cfg.vocab:
            raise ValueError(f"logits shape {tuple(logits.shape)} does not match the context")
        if logits.stride(3) != 1:
            raise ValueError("the vocabulary axis of logits must be contiguous")
        if _dtype_code(logits.dtype) != self.cfg.dtype:
            raise ValueError("logits dtype does not match the context")
        a = cos_verify_args()
        a.logits = logits.data_ptr()
        a.stride_model, a.stride_row, a.stride_pos = logits.stride(0), logits.stride(1), logits.stride(2)
        a.draft_tokens = drafts.data_ptr() if (drafts is not None and drafts.numel() > 0) else None
        a.proposer = proposer.data_ptr()
        a.batch, a.flags, a.row_base = B, flags, row_base
        a.seed, a.offset = seed & 0xFFFFFFFFFFFFFFFF, offset & 0xFFFFFFFFFFFFFFFF
        a.accept_count = outs["accept_count"].data_ptr()
        a.out_tokens = outs["out_tokens"].data_ptr()
        a.row_status = outs["row_status"].data_ptr()
        a.diag = outs["diag"].data_ptr() if "diag" in outs else None
        a.dump_r = outs["r"].data_ptr() if "r" in outs else None
        a.bonus_prob = outs["bonus_prob"].data_ptr() if "bonus_prob" in outs else None
        a.bonus_model = bonus_model if (bonus_model is not None and bonus_model >= 0) else 0
        a.offset_device = offset_device.data_ptr() if offset_device is not None else None
        a.lse = outs["lse"].data_ptr() if "lse" in outs else None
        return a

    def set_one_launch(self, enable=True):
        """cos_verify_set_one_launch: 1 / True: later runs take the one-launch kernel; 2: staged streaming launch, tokens
        drawn by that kernel's drawing items; 0: the staged launches (raises if the configuration is not covered)."""
        self._check(self._lib.cos_verify_set_one_launch(self._ctx, int(enable)))

    def set_wait_limit(self, polls: int, test_drop_report: bool = False):
        """cos_verify_set_wait_limit: bound of the kernel's internal polls (and the test hook that makes one run out)."""
        self._check(self._lib.cos_verify_set_wait_limit(self._ctx, int(polls), int(bool(test_drop_report))))

    def set_stage_timing(self, enable: bool):
        """cos_verify_set_stage_timing: record events around every launch of later runs."""
        self._check(self._lib.cos_verify_set_stage_timing(self._ctx, int(bool(enable))))

    def stage_ms(self):
        """cos_verify_get_stage_ms: durations (ms) of the launches of the last timed run."""
        ms = (ctypes.c_float * 4)()
        count = ctypes.c_int32(0)
        self._check(self._lib.cos_verify_get_stage_ms(self._ctx, ms, ctypes.byref(count)))
        return [float(ms[k]) for k in range(count.value)]

    @staticmethod
    def _alloc_outs(B, P, V, device, diag, dump_r, pin=False):
        import torch
        kw = dict(device=device)
        if pin:
            kw["pin_memory"] = True
        outs = {
            "accept_count": torch.empty(B, dtype=torch.int32, **kw),
            "out_tokens": torch.empty((B, P), dtype=torch.int32, **kw),
            "row_status": torch.empty(B, dtype=torch.int32, **kw),
            "bonus_prob": torch.empty(B, dtype=torch.float32, **kw),
        }
        if diag:
            outs["diag"] = torch.empty((B, P, 4), dtype=torch.float32, **kw)
        if dump_r:
            outs["r"] = torch.empty((B, P, V), dtype=torch.float32, **kw)
        return outs

    # -- the calls -------------------------------------------------------------------
    def run(self, logits, drafts, proposer, seed: int, offset: int, row_base: int = 0, flags: int = 0,
            diag: bool = False, dump_r: bool = False, outs: Optional[dict] = None, stream=None,
            bonus_model: Optional[int] = None, offset_device=None, lse: bool = False) -> dict:
        """cos_verify_run on device tensors; asynchronous on `stream` (default: torch's current stream).

        `proposer` is [B], or [B, gamma+1] to name the proposer of every draft (Algorithm 2); `bonus_model`
        draws the token after gamma acceptances from that model's own distribution (Sec. 3.3).  The outputs
        include "bonus_prob" [B]: the bonus token's probability under the law it was drawn from.
        `offset_device` (a one-element int64 device tensor) replaces `offset`: the kernels read it, so a
        run captured in a CUDA graph can be replayed with a new offset each time."""
        import torch
        if not logits.is_cuda:
            raise ValueError("run() needs device tensors; use run_host() for host tensors")
        for t, name in ((drafts, "drafts"), (proposer, "proposer")):
            if t is not None and t.numel() > 0 and (t.dtype != torch.int32 or not t.is_contiguous() or not t.is_cuda):
                raise ValueError(f"{name} must be a contiguous int32 device tensor")
        n, B, P, V = logits.shape
        if outs is None:
            outs = self._alloc_outs(B, P, V, logits.device, diag, dump_r)
            if lse:     # log-sum-exp behind every softmax of a position: [B, gamma+1, n] (ensemble) or [B, gamma+1, 2]
                slots = self.cfg.n if self.cfg.combine == COS_COMBINE_PROB_ENSEMBLE else 2
                outs["lse"] = torch.empty((B, P, slots), dtype=torch.float32, device=logits.device)
        if offset_device is not None and (offset_device.dtype != torch.int64 or not offset_device.is_cuda):
            raise ValueError("offset_device must be an int64 device tensor")
        a = self._fill_args(logits, drafts, proposer, seed, offset, row_base, flags, outs, bonus_model, offset_device)
        s = torch.cuda.current_stream(logits.device) if stream is None else stream
        self._check(self._lib.cos_verify_run(self._ctx, ctypes.byref(a), ctypes.c_void_p(s.cuda_stream)))
        return outs

    def run_host(self, logits, drafts, proposer, seed: int, offset: int, row_base: int = 0, flags: int = 0,
                 diag: bool = False, outs: Optional[dict] = None, stream=None,
                 bonus_model: Optional[int] = None) -> dict:
        """cos_verify_run_host on host tensors: copies in, runs, copies out, waits."""
        import torch
        if logits.is_cuda or not logits.is_contiguous():
            raise ValueError("run_host() needs contiguous host tensors")
        for t, name in ((drafts, "drafts"), (proposer, "proposer")):
            if t is not None and t.numel() > 0 and (t.dtype != torch.int32 or not t.is_contiguous() or t.is_cuda):
                raise ValueError(f"{name} must be a contiguous int32 host tensor")
        n, B, P, V = logits.shape
        if outs is None:
            outs = self._alloc_outs(B, P, V, "cpu", diag, False, pin=True)
        a = self._fill_args(logits, drafts, proposer, seed, offset, row_base, flags, outs, bonus_model)
        s = torch.cuda.current_stream(self.cfg.device) if stream is None else stream
        self._check(self._lib.cos_verify_run_host(self._ctx, ctypes.byref(a), ctypes.c_void_p(s.cuda_stream)))
        return outs

    def close(self):
        if getattr(self, "_ctx", None) is not None and self._ctx.value:
            self._lib.cos_verify_destroy(self._ctx)
            self._ctx = ctypes.c_void_p()

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()


def measure_ceiling(kind: int, buf, reps: int = 10, stream=None) -> float:
    """cos_verify_measure_ceiling: GB/s of a read-only streaming pass over the device tensor `buf` (kind 0), or of
    the same pass with one fast exponential per 16-bit entry (kind 1)."""
    import torch
    lib = load_library()
    out = torch.empty(1024 * torch.cuda.get_device_properties(buf.device).multi_processor_count, dtype=torch.float32,
                      device=buf.device)
    ms = ctypes.c_float(0.0)
    nbytes = buf.numel() * buf.element_size()
    s = torch.cuda.current_stream(buf.device) if stream is None else stream
    with torch.cuda.device(buf.device):
        st = lib.cos_verify_measure_ceiling(kind, buf.data_ptr(), nbytes, out.data_ptr(), out.numel(), reps,
                                            ctypes.byref(ms), ctypes.c_void_p(s.cuda_stream))
    if st != COS_OK:
        raise CosVerifyError(st, "cos_verify_measure_ceiling")
    return nbytes / (ms.value * 1e-3) / 1e9


def run_static(n: int, combine: int, weights: Sequence[float], temperature: float, gamma: int, vocab: int,
               logits, drafts, proposer, seed: int, offset: int, mask_model: int = -1, mask_alpha: float = 1.0,
               device: int = 0, cluster_size: int = 0, row_base: int = 0, flags: int = 0, outs: dict = None,
               stream=None, bonus_model: Optional[int] = None) -> dict:
    """cos_verify_run_static: one verification pass with no context and no device allocation.

    For hosts that cannot call cudaMalloc where they verify (a device fully owned by an engine's
    memory pool, or a serving loop that must avoid the device-wide stall of cudaMalloc/cudaFree):
    the kernel's scratch is an array built into the library.  `outs` must hold the preallocated
    output tensors ("accept_count" [B], "out_tokens" [B, gamma+1], "row_status" [B], all int32,
    optionally "diag" [B, gamma+1, 4] float32) so that this wrapper allocates nothing either.
    Limits: B <= 1024 and B * (gamma + 1) <= 8192.  Calls share the built-in array, so calls
    that overlap on the GPU race; order them on one stream.
    """
    import torch
    lib = load_library()
    lib.cos_verify_run_static.argtypes = [ctypes.POINTER(cos_verify_config), ctypes.POINTER(cos_verify_args),
                                          ctypes.c_void_p]
    lib.cos_verify_run_static.restype = ctypes.c_int
    cfg = cos_verify_config()
    cfg.n, cfg.combine = n, combine
    for i, w in enumerate(list(weights)[:COS_MAX_MODELS]):
        cfg.weights[i] = w
    cfg.mask_model, cfg.mask_alpha, cfg.temperature = mask_model, mask_alpha, temperature
    cfg.gamma, cfg.vocab, cfg.max_batch = gamma, vocab, logits.shape[1]
    cfg.dtype, cfg.device, cfg.cluster_size, cfg.host_staging = _dtype_code(logits.dtype), device, cluster_size, 0
    if outs is None:
        raise ValueError("run_static needs preallocated outputs (it must not allocate)")
    a = cos_verify_args()
    a.logits = logits.data_ptr()
    a.stride_model, a.stride_row, a.stride_pos = logits.stride(0), logits.stride(1), logits.stride(2)
    a.draft_tokens = drafts.data_ptr() if (drafts is not None and drafts.numel() > 0) else None
    a.proposer = proposer.data_ptr()
    if proposer.dim() == 2:
        flags |= COS_RUN_PROPOSER_PER_POSITION
    if bonus_model is not None and bonus_model >= 0:
        flags |= COS_RUN_BONUS_FROM_MODEL
    a.batch, a.flags, a.row_base = logits.shape[1], flags, row_base
    a.seed, a.offset = seed & 0xFFFFFFFFFFFFFFFF, offset & 0xFFFFFFFFFFFFFFFF
    a.accept_count = outs["accept_count"].data_ptr()
    a.out_tokens = outs["out_tokens"].data_ptr()
    a.row_status = outs["row_status"].data_ptr()
    a.diag = outs["diag"].data_ptr() if "diag" in outs else None
    a.dump_r = None
    a.bonus_prob = outs["bonus_prob"].data_ptr() if "bonus_prob" in outs else None
    a.bonus_model = bonus_model if (bonus_model is not None and bonus_model >= 0) else 0
    s = torch.cuda.current_stream(logits.device) if stream is None else stream
    st = lib.cos_verify_run_static(ctypes.byref(cfg), ctypes.byref(a), ctypes.c_void_p(s.cuda_stream))
    if st != COS_OK:
        raise CosVerifyError(st, lib.cos_verify_last_error(None).decode())
    return outs
