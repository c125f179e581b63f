"""Seeded synthetic region-marker traces (input generator; none of the method's arithmetic).

The traces stand in for recorded traces of the workloads the paper profiles (Section 4: a
warp-specialised persistent GEMM, attention kernels, a persistent decode megakernel), which
need instrumented kernels and a tracer that are not available. The same C++ source is built for
the host (threads over streams) and for the device (one thread per stream); both write
bit-identical events, so a CPU checker can regenerate any stream of a trace that was generated
in GPU memory.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, replace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))

EVENT_DTYPE = np.dtype([("ts", "<u8"), ("tag", "<u4"), ("ctx", "<u4")])

TINY, GEMM, ATTENTION, DECODE = 1, 2, 3, 4
BASE_SEED = 2609122990


class _Params(ctypes.Structure):
    _fields_ = [
        ("kind", ctypes.c_uint32),
        ("num_ctas", ctypes.c_uint32),
        ("iters", ctypes.c_uint32),
        ("inner", ctypes.c_uint32),
        ("seed", ctypes.c_uint64),
        ("thr_dup_begin", ctypes.c_uint64),
        ("thr_drop_end", ctypes.c_uint64),
        ("thr_trunc", ctypes.c_uint64),
    ]


def _threshold(p: float) -> int:
    if p <= 0.0:
        return 0
    return min(int(p * 2.0**64), 2**64 - 1)


@dataclass(frozen=True)
class TraceSpec:
    """One synthetic trace. `iters`/`inner` mean: TINY events per stream / unused; GEMM tile
    iterations / unused; ATTENTION tiles / KV iterations per tile; DECODE tokens / layers."""

    kind: int
    num_ctas: int
    iters: int
    inner: int = 0
    seed: int = BASE_SEED
    p_dup_begin: float = 0.0
    p_drop_end: float = 0.0
    p_trunc: float = 0.0
    name: str = ""

    @property
    def warps_per_cta(self) -> int:
        return {TINY: 4, GEMM: 12}.get(self.kind, 16)

    @property
    def num_streams(self) -> int:
        return self.num_ctas * self.warps_per_cta

    @property
    def num_regions(self) -> int:
        return {TINY: 8, GEMM: 5, ATTENTION: 9}.get(self.kind, 4 + 9 * self.inner)

    @property
    def num_sms(self) -> int:
        return max(1, self.num_ctas // 2) if self.kind == TINY else self.num_ctas

    @property
    def cta_sm(self) -> np.ndarray:
        c = np.arange(self.num_ctas, dtype=np.uint32)
        return (c // 2).astype(np.uint32) if self.kind == TINY and self.num_ctas > 1 else c

    @property
    def overlap_pairs(self) -> np.ndarray:
        pairs = {
            TINY: [(0, 1), (2, 3), (1, 1)],
            GEMM: [(1, 2)],          # tma_load vs mma
            ATTENTION: [(2, 3)],     # load_KV vs qk_mma
            DECODE: [(4 + 1, 4 + 3)],  # qkv vs attn of layer 0
        }[self.kind]
        return np.asarray(pairs, dtype=np.uint32)

    @property
    def well_formed(self) -> bool:
        return self.p_dup_begin == 0 and self.p_drop_end == 0 and self.p_trunc == 0

    def _c(self) -> _Params:
        return _Params(self.kind, self.num_ctas, self.iters, self.inner, self.seed,
                       _threshold(self.p_dup_begin), _threshold(self.p_drop_end), _threshold(self.p_trunc))

    def scaled(self, num_ctas: int | None = None, iters: int | None = None) -> "TraceSpec":
        return replace(self, num_ctas=num_ctas or self.num_ctas, iters=iters or self.iters)


def config(index: int) -> TraceSpec:
    """The five benchmark configurations at full size (index 0..4)."""
    if index == 0:
        return TraceSpec(TINY, 4, 626, 0, BASE_SEED + 0, name="tiny")
    if index == 1:
        return TraceSpec(GEMM, 148, 2000, 0, BASE_SEED + 1, name="persistent_gemm")
    if index == 2:
        return TraceSpec(ATTENTION, 148, 22, 512, BASE_SEED + 2, name="attention")
    if index == 3:
        return TraceSpec(DECODE, 148, 256, 22, BASE_SEED + 3, name="decode_megakernel")
    if index == 4:
        return TraceSpec(GEMM, 148, 2000, 0, BASE_SEED + 4, 0.0005, 0.001, 0.01, name="malformed_gemm")
    raise ValueError("config index must be 0..4")


_host = None
_cuda = None


def _host_lib():
    global _host
    if _host is None:
        path = os.path.join(_HERE, "libtracegen_host.so")
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: run `python -c 'import __graft_entry__ as g; g.build()'`")
        lib = ctypes.CDLL(path)
        lib.tg_lengths.argtypes = [ctypes.POINTER(_Params), ctypes.c_void_p, ctypes.c_int]
        lib.tg_lengths.restype = ctypes.c_int
        lib.tg_fill.argtypes = [ctypes.POINTER(_Params), ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32,
                                ctypes.c_void_p, ctypes.c_int]
        lib.tg_fill.restype = ctypes.c_int
        _host = lib
    return _host


def _cuda_lib():
    global _cuda
    if _cuda is None:
        path = os.path.join(_HERE, "libtracegen_cuda.so")
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: run `python -c 'import __graft_entry__ as g; g.build()'`")
        lib = ctypes.CDLL(path)
        lib.tg_cuda_lengths.argtypes = [ctypes.POINTER(_Params), ctypes.c_void_p, ctypes.c_void_p]
        lib.tg_cuda_lengths.restype = ctypes.c_int
        lib.tg_cuda_fill.argtypes = [ctypes.POINTER(_Params), ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32,
                                     ctypes.c_void_p, ctypes.c_void_p]
        lib.tg_cuda_fill.restype = ctypes.c_int
        _cuda = lib
    return _cuda


def default_threads() -> int:
    return max(1, len(os.sched_getaffinity(0)))


def host_offsets(spec: TraceSpec, nthreads: int | None = None) -> np.ndarray:
    """CSR stream offsets [S+1] (uint64) of the trace."""
    lens = np.zeros(spec.num_streams, dtype=np.uint64)
    p = spec._c()
    rc = _host_lib().tg_lengths(ctypes.byref(p), lens.ctypes.data, nthreads or default_threads())
    assert rc == 0
    offs = np.zeros(spec.num_streams + 1, dtype=np.uint64)
    np.cumsum(lens, out=offs[1:])
    return offs


def host_streams(spec: TraceSpec, offsets: np.ndarray, s_lo: int, s_hi: int, nthreads: int | None = None) -> np.ndarray:
    """Events of streams [s_lo, s_hi) as one structured array (stream s_lo first)."""
    n = int(offsets[s_hi] - offsets[s_lo])
    ev = np.zeros(n, dtype=EVENT_DTYPE)
    p = spec._c()
    offs = np.ascontiguousarray(offsets, dtype=np.uint64)
    rc = _host_lib().tg_fill(ctypes.byref(p), offs.ctypes.data, s_lo, s_hi, ev.ctypes.data, nthreads or default_threads())
    assert rc == 0
    return ev


def generate_host(spec: TraceSpec, nthreads: int | None = None):
    """(events structured array [N], stream_offsets uint64 [S+1]) in host memory."""
    offs = host_offsets(spec, nthreads)
    return host_streams(spec, offs, 0, spec.num_streams, nthreads), offs


def generate_cuda(spec: TraceSpec, device="cuda:0"):
    """(events uint8 tensor [N*16], stream_offsets int64 tensor [S+1]) in device memory,
    bit-identical to generate_host()."""
    import torch

    lib = _cuda_lib()
    dev = torch.device(device)
    p = spec._c()
    S = spec.num_streams
    with torch.cuda.device(dev):
        stream = torch.cuda.current_stream().cuda_stream
        if spec.p_dup_begin == 0 and spec.p_drop_end == 0:
            offs = torch.from_numpy(host_offsets(spec).astype(np.int64)).to(dev)
        else:
            lens = torch.zeros(S, dtype=torch.int64, device=dev)
            rc = lib.tg_cuda_lengths(ctypes.byref(p), lens.data_ptr(), stream)
            if rc != 0:
                raise RuntimeError(f"tg_cuda_lengths: CUDA error {rc}")
            offs = torch.zeros(S + 1, dtype=torch.int64, device=dev)
            offs[1:] = torch.cumsum(lens, 0)
        n = int(offs[-1].item())
        events = torch.empty(max(n, 1) * 16, dtype=torch.uint8, device=dev)[: n * 16]
        rc = lib.tg_cuda_fill(ctypes.byref(p), offs.data_ptr(), 0, S, events.data_ptr(), stream)
        if rc != 0:
            raise RuntimeError(f"tg_cuda_fill: CUDA error {rc}")
        torch.cuda.synchronize(dev)
    return events, offs
