"""Thin ctypes binding of librtprune.so: argument marshalling only.

The names mirror include/rtprune.h.  torch is used for device memory and streams; every step of the
pruning path runs in the library's CUDA kernels.  There is no CPU fallback: if the library cannot be
loaded, or no CUDA device is present, the calls raise.
"""
from __future__ import annotations

import ctypes
import numpy as np
import os
from dataclasses import dataclass
from typing import Optional

import torch

from . import build as _build

STATS_STRIDE = 8
BF16, FP32 = 0, 1
SINKHORN_AUTO, SINKHORN_LOG, SINKHORN_SCALING, SINKHORN_EXACT = 0, 1, 2, 3
SCHEDULE_AUTO, SCHEDULE_SEPARATE, SCHEDULE_FUSED = 0, 1, 2
DEV_NONFINITE, DEV_TIMEOUT, DEV_BAD_OFFSETS = 1, 2, 4

STATUS_NAMES = {0: "RTPRUNE_OK", 1: "RTPRUNE_ERR_INVALID_ARG", 2: "RTPRUNE_ERR_UNSUPPORTED",
                3: "RTPRUNE_ERR_WORKSPACE", 4: "RTPRUNE_ERR_CUDA", 5: "RTPRUNE_ERR_NONFINITE",
                6: "RTPRUNE_ERR_TIMEOUT", 7: "RTPRUNE_ERR_BAD_OFFSETS"}


class RtpruneError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s returned %s" % (where, STATUS_NAMES.get(status, status)))


class CParams(ctypes.Structure):
    """rtprune_params_t."""
    _fields_ = [("dynamic", ctypes.c_int32), ("r_fixed", ctypes.c_float),
                ("rho", ctypes.c_void_p), ("phi_lo", ctypes.c_float), ("phi_hi", ctypes.c_float),
                ("r_max", ctypes.c_float), ("z", ctypes.c_float), ("alpha", ctypes.c_float),
                ("eps", ctypes.c_float), ("iters", ctypes.c_int32), ("form", ctypes.c_int32),
                ("stop_at_fixed_point", ctypes.c_int32), ("tol", ctypes.c_float),
                ("criterion", ctypes.c_int32), ("schedule", ctypes.c_int32)]


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """Loads (building first if the sources are newer) the C-ABI library.  Raises on failure."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if _build.stale():
        path = _build.build()
    if not os.path.exists(path):
        raise RuntimeError("librtprune.so is missing and could not be built")
    L = ctypes.CDLL(path)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    pp = ctypes.POINTER(CParams)
    L.rtprune_default_params.argtypes = [pp]
    L.rtprune_plan.argtypes = [ctypes.POINTER(vp), i32, ctypes.c_int, i32, i64, i32,
                               ctypes.POINTER(sz)]
    L.rtprune_run.argtypes = [vp, vp, vp, vp, i32, i64, pp, vp, sz, vp, vp, vp, vp, vp, vp, vp, vp]
    L.rtprune_workspace_init.argtypes = [vp, vp, vp, sz]
    L.rtprune_select.argtypes = [vp, vp, vp, vp, i32, i64, pp, vp, sz, vp, vp, vp, vp, vp]
    L.rtprune_select_static.argtypes = [vp, vp, vp, vp, i32, i64, pp, vp, vp, vp, vp, vp]
    L.rtprune_static_scratch_needed.argtypes = [vp, ctypes.POINTER(sz)]
    L.rtprune_query_status_static.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    L.rtprune_test_expire_waits.argtypes = [vp, vp, vp, sz, ctypes.c_uint32, vp]
    L.rtprune_test_set_poll_limit.argtypes = [vp, ctypes.c_int64]
    L.rtprune_run_host.argtypes = [vp, vp, vp, vp, vp, i32, i64, pp, vp, sz,
                                   vp, vp, vp, vp, vp, vp, vp, vp]
    L.rtprune_host_arena_bytes.argtypes = [vp, ctypes.POINTER(sz)]
    L.rtprune_query_status.argtypes = [vp, vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    L.rtprune_density.argtypes = [vp, vp, i32, i32, i32, i32, ctypes.c_float, vp, vp, vp]
    L.rtprune_profile_enable.argtypes = [vp, i32]
    L.rtprune_profile_read.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_float),
                                       ctypes.POINTER(ctypes.c_char_p)]
    L.rtprune_last_launch_count.argtypes = [vp]
    L.rtprune_last_cuda_error.argtypes = [vp]
    L.rtprune_last_host_ns.argtypes = [vp]
    L.rtprune_last_host_ns.restype = ctypes.c_int64
    L.rtprune_destroy.argtypes = [vp]
    L.rtprune_destroy.restype = None
    L.rtprune_status_string.argtypes = [ctypes.c_int]
    L.rtprune_status_string.restype = ctypes.c_char_p
    L.rtprune_version.restype = i32
    _lib = L
    return L


def _check(status: int, where: str) -> None:
    if status != 0:
        raise RtpruneError(status, where)


def default_params() -> CParams:
    p = CParams()
    _check(lib().rtprune_default_params(ctypes.byref(p)), "rtprune_default_params")
    return p


def make_params(rho: Optional[torch.Tensor] = None, **kw) -> CParams:
    """Paper defaults overridden by keyword (field names of rtprune_params_t)."""
    p = default_params()
    for k, v in kw.items():
        if not hasattr(p, k) or k == "rho":
            raise KeyError(k)
        setattr(p, k, v)
    p.rho = rho.data_ptr() if rho is not None else None
    return p


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _stream_handle(stream: Optional[torch.cuda.Stream]):
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


@dataclass
class Outputs:
    """Device (or pinned host) tensors the library fills; see rtprune_run in rtprune.h."""
    Y: torch.Tensor
    out_offsets: torch.Tensor
    counts: torch.Tensor
    kept_idx: torch.Tensor
    merged_idx: torch.Tensor
    merge_partner: torch.Tensor
    merge_weight: torch.Tensor
    stats: torch.Tensor

    @staticmethod
    def allocate(total_tokens: int, batch: int, d: int, dtype: torch.dtype, device,
                 pin: bool = False) -> "Outputs":
        kw = dict(device=device, pin_memory=pin) if pin else dict(device=device)
        n = max(total_tokens, 1)
        return Outputs(
            Y=torch.empty((n, d), dtype=dtype, **kw),
            out_offsets=torch.zeros(batch + 1, dtype=torch.int32, **kw),
            counts=torch.zeros(max(batch, 1), dtype=torch.int32, **kw),
            kept_idx=torch.full((n,), -1, dtype=torch.int32, **kw),
            merged_idx=torch.full((n,), -1, dtype=torch.int32, **kw),
            merge_partner=torch.full((n,), -1, dtype=torch.int32, **kw),
            merge_weight=torch.zeros(n, dtype=torch.float32, **kw),
            stats=torch.zeros((max(batch, 1), STATS_STRIDE), dtype=torch.float32, **kw))


class Plan:
    """rtprune_plan_t plus a torch-allocated workspace on the current device."""

    def __init__(self, d: int, dtype: torch.dtype, max_batch: int, max_total_tokens: int,
                 max_tokens_per_image: int, device: Optional[torch.device] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("rtprune needs a CUDA device; there is no CPU path")
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else device
        self.d, self.dtype = d, dtype
        self.max_batch, self.max_total, self.max_tokens = max_batch, max_total_tokens, max_tokens_per_image
        code = {torch.bfloat16: BF16, torch.float32: FP32}[dtype]
        h = ctypes.c_void_p()
        ws = ctypes.c_size_t()
        with torch.cuda.device(self.device):
            _check(lib().rtprune_plan(ctypes.byref(h), d, code, max_batch, max_total_tokens,
                                      max_tokens_per_image, ctypes.byref(ws)), "rtprune_plan")
            self.handle = h
            self.workspace_bytes = ws.value
            self.workspace = torch.empty(ws.value, dtype=torch.uint8, device=self.device)
            assert self.workspace.data_ptr() % 256 == 0
            self.workspace_init()
        self._arena = None

    # -- rtprune_workspace_init
    def workspace_init(self, stream: Optional[torch.cuda.Stream] = None) -> None:
        _check(lib().rtprune_workspace_init(self.handle, _stream_handle(stream),
                                            self.workspace.data_ptr(), self.workspace_bytes),
               "rtprune_workspace_init")

    # -- rtprune_run
    def run(self, X: torch.Tensor, offsets: torch.Tensor, params: CParams, out: Outputs,
            stream: Optional[torch.cuda.Stream] = None) -> None:
        batch = offsets.numel() - 1
        _check(lib().rtprune_run(self.handle, _stream_handle(stream), X.data_ptr(),
                                 offsets.data_ptr(), batch, X.shape[0], ctypes.byref(params),
                                 self.workspace.data_ptr(), self.workspace_bytes, out.Y.data_ptr(),
                                 out.out_offsets.data_ptr(), out.counts.data_ptr(),
                                 out.kept_idx.data_ptr(), out.merged_idx.data_ptr(),
                                 out.merge_partner.data_ptr(), out.merge_weight.data_ptr(),
                                 out.stats.data_ptr()), "rtprune_run")

    # -- rtprune_select
    def select(self, X: torch.Tensor, offsets: torch.Tensor, params: CParams, out: Outputs,
               norms_out: Optional[torch.Tensor] = None, order_out: Optional[torch.Tensor] = None,
               stream: Optional[torch.cuda.Stream] = None) -> None:
        batch = offsets.numel() - 1
        _check(lib().rtprune_select(self.handle, _stream_handle(stream), X.data_ptr(),
                                    offsets.data_ptr(), batch, X.shape[0], ctypes.byref(params),
                                    self.workspace.data_ptr(), self.workspace_bytes,
                                    out.out_offsets.data_ptr(), out.counts.data_ptr(),
                                    out.stats.data_ptr(), _ptr(norms_out), _ptr(order_out)),
               "rtprune_select")

    # -- rtprune_select_static
    def select_static(self, X: torch.Tensor, offsets: torch.Tensor, params: CParams, out: Outputs,
                      norms_out: Optional[torch.Tensor] = None,
                      order_out: Optional[torch.Tensor] = None,
                      stream: Optional[torch.cuda.Stream] = None) -> None:
        """Stage 1 on the library's built-in scratch array: nothing is allocated by the call."""
        batch = offsets.numel() - 1
        _check(lib().rtprune_select_static(self.handle, _stream_handle(stream), X.data_ptr(),
                                           offsets.data_ptr(), batch, X.shape[0],
                                           ctypes.byref(params), out.out_offsets.data_ptr(),
                                           out.counts.data_ptr(), out.stats.data_ptr(),
                                           _ptr(norms_out), _ptr(order_out)),
               "rtprune_select_static")

    # -- rtprune_static_scratch_needed / rtprune_query_status_static
    def static_scratch_needed(self) -> int:
        n = ctypes.c_size_t()
        _check(lib().rtprune_static_scratch_needed(self.handle, ctypes.byref(n)), "rtprune_static_scratch_needed")
        return n.value

    def query_status_static(self, stream: Optional[torch.cuda.Stream] = None) -> int:
        """Synchronises, returns the status bits the last select_static call left (0 = clean), clears them."""
        flags = ctypes.c_uint32()
        lib().rtprune_query_status_static(self.handle, _stream_handle(stream), ctypes.byref(flags))
        return flags.value

    # -- rtprune_test_expire_waits
    def expire_waits(self, poll_limit: int, stream: Optional[torch.cuda.Stream] = None) -> int:
        """Test aid: lets two bounded device-side waits run out on this plan's workspace; returns how many did."""
        expired = torch.zeros(1, dtype=torch.int32, device=self.device)
        _check(lib().rtprune_test_expire_waits(self.handle, _stream_handle(stream), self.workspace.data_ptr(),
                                               self.workspace.numel(), int(poll_limit), expired.data_ptr()),
               "rtprune_test_expire_waits")
        return int(expired.item())

    def set_poll_limit(self, polls: int) -> None:
        """Test aid: polls after which stage 1's waits on its copies give up (negative: the default)."""
        _check(lib().rtprune_test_set_poll_limit(self.handle, int(polls)), "rtprune_test_set_poll_limit")

    # -- rtprune_host_arena_bytes / rtprune_run_host
    def host_arena_bytes(self) -> int:
        n = ctypes.c_size_t()
        _check(lib().rtprune_host_arena_bytes(self.handle, ctypes.byref(n)), "rtprune_host_arena_bytes")
        return n.value

    def run_host(self, X: torch.Tensor, offsets: torch.Tensor, rho: Optional[torch.Tensor],
                 params: CParams, out: Outputs, stream: Optional[torch.cuda.Stream] = None) -> None:
        """Host tensors in (pinned for speed), host tensors out; asynchronous on the stream."""
        if self._arena is None:
            self._arena = torch.empty(self.host_arena_bytes(), dtype=torch.uint8, device=self.device)
        for t in (X, offsets, out.Y, out.out_offsets):
            assert t.device.type == "cpu"
        batch = offsets.numel() - 1
        _check(lib().rtprune_run_host(self.handle, _stream_handle(stream), X.data_ptr(),
                                      offsets.data_ptr(), _ptr(rho), batch, X.shape[0],
                                      ctypes.byref(params), self._arena.data_ptr(),
                                      self._arena.numel(), out.Y.data_ptr(),
                                      out.out_offsets.data_ptr(), out.counts.data_ptr(),
                                      out.kept_idx.data_ptr(), out.merged_idx.data_ptr(),
                                      out.merge_partner.data_ptr(), out.merge_weight.data_ptr(),
                                      out.stats.data_ptr()), "rtprune_run_host")

    # -- rtprune_query_status
    def query_status(self, stream: Optional[torch.cuda.Stream] = None, workspace=None) -> int:
        """Synchronises, returns the raw device status bits (0 = clean) and clears them."""
        flags = ctypes.c_uint32()
        ws = self.workspace.data_ptr() if workspace is None else workspace
        lib().rtprune_query_status(self.handle, _stream_handle(stream), ws, ctypes.byref(flags))
        return flags.value

    # -- rtprune_profile_enable / rtprune_profile_read
    def profile_enable(self, enable: bool = True) -> None:
        _check(lib().rtprune_profile_enable(self.handle, int(enable)), "rtprune_profile_enable")

    def profile_read(self):
        """[(kernel name, milliseconds)] of the most recent run (waits for it)."""
        n = ctypes.c_int32()
        ms = (ctypes.c_float * 8)()
        names = (ctypes.c_char_p * 8)()
        _check(lib().rtprune_profile_read(self.handle, ctypes.byref(n), ms, names),
               "rtprune_profile_read")
        return [(names[i].decode(), float(ms[i])) for i in range(n.value)]

    @property
    def last_launch_count(self) -> int:
        return lib().rtprune_last_launch_count(self.handle)

    @property
    def last_host_ns(self) -> int:
        return lib().rtprune_last_host_ns(self.handle)

    @property
    def last_cuda_error(self) -> int:
        return lib().rtprune_last_cuda_error(self.handle)

    def close(self) -> None:
        if getattr(self, "handle", None):
            lib().rtprune_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def density(images: torch.Tensor, patch: int = 64, tau: float = 0.2, *, want_patch_counts: bool = False,
            stream: Optional[torch.cuda.Stream] = None):
    """rtprune_density: textual density rho [batch] (float32, on the images' device) of a batch of page
    images [batch, H, W, 3] uint8 (Eq. 9).  Returns (rho, image_counts, edge_counts or None)."""
    if images.dtype != torch.uint8 or images.dim() != 4 or images.shape[3] != 3 or not images.is_contiguous():
        raise ValueError("images must be a contiguous [batch, H, W, 3] uint8 tensor")
    if not images.is_cuda:
        raise ValueError("images must live on a CUDA device")
    batch, H, W, _ = images.shape
    dev = images.device
    rho = torch.empty(batch, dtype=torch.float32, device=dev)
    counts = torch.empty(batch, dtype=torch.int32, device=dev)          # uint32 in the library
    per_patch = None
    if want_patch_counts and patch > 0:
        per_patch = torch.empty((batch, H // patch, W // patch), dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        _check(lib().rtprune_density(_stream_handle(stream), images.data_ptr(), batch, H, W, patch, float(tau),
                                     rho.data_ptr(), counts.data_ptr(), _ptr(per_patch)), "rtprune_density")
    return rho, counts, per_patch


def shard_images(batch: int, world_size: int, rank: int):
    """Contiguous range of images [lo, hi) owned by `rank`: images are independent, so a multi-GPU
    run is this split with no exchange."""
    base, extra = divmod(batch, world_size)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def shard_images_by_tokens(offsets, world_size: int, rank: int):
    """Contiguous range of images [lo, hi) for `rank` on a ragged batch, balanced by work instead of by count:
    the cut before rank k is the image boundary nearest to k / world_size of the batch's cost, an image of N
    tokens costing N (the streaming passes) + N^2 / 1600 (scores, Sinkhorn and merge grow with M B <= N^2 / 4;
    the weight makes the two terms equal at 400 tokens).  Every rank computes the same cuts from the offsets."""
    offsets = np.asarray(offsets, dtype=np.int64)
    n = np.diff(offsets).astype(np.float64)
    cost = np.concatenate([[0.0], np.cumsum(n + n * n / 1600.0)])
    total = cost[-1]
    cuts = [0]
    for k in range(1, world_size):
        j = int(np.argmin(np.abs(cost - total * k / world_size)))
        cuts.append(max(j, cuts[-1]))
    cuts.append(len(n))
    return cuts[rank], cuts[rank + 1]


def shard_slice(offsets, world_size: int, rank: int, *, by_tokens: bool = False):
    """What `rank` takes of a ragged batch: (lo, hi) its images, (row_lo, row_hi) its rows of X, and its own
    offsets array, rebased so that it starts at 0 (what rtprune_run expects for the slice).  by_tokens: balance
    the ranks by work (shard_images_by_tokens) instead of by image count."""
    offsets = np.asarray(offsets, dtype=np.int64)
    lo, hi = (shard_images_by_tokens(offsets, world_size, rank) if by_tokens
              else shard_images(len(offsets) - 1, world_size, rank))
    row_lo, row_hi = int(offsets[lo]), int(offsets[hi])
    return (lo, hi), (row_lo, row_hi), (offsets[lo:hi + 1] - row_lo).astype(np.int32)


def packed_row_base(kept_rows_of_ranks, rank: int) -> int:
    """Rows of the packed output that the lower ranks produce: what a rank adds to its local out_offsets to get
    the positions its images have in the output of the whole batch."""
    return int(sum(int(c) for c in list(kept_rows_of_ranks)[:rank]))


def global_out_offsets(local_out_offsets: torch.Tensor, group=None) -> torch.Tensor:
    """The rank's out_offsets in the numbering of the whole batch.  The only datum that crosses ranks is each
    rank's number of kept rows (one all_gather of a scalar; nothing on the data path).  With no process group
    initialised the local offsets are returned as they are."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return local_out_offsets.clone()
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    mine = local_out_offsets[-1:].to(torch.int64).clone()
    every = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(every, mine, group=group)
    return local_out_offsets + packed_row_base([int(t.item()) for t in every], rank)

