"""Synthetic mapping-run traces (input generator only): a marker trace with "PC p executed k times"
records inserted after every begin marker, in the marker encoding of include/argus.h (a begin/end
pair of the extra region id R with ctx = PC index and ts 0 / k). Stands in for the instrumented
mapping run of the paper's PC-to-region attribution (static PC counts of its megakernel study:
43,856 to 70,560). Plain tensor operations; works on CPU and CUDA tensors alike."""
from __future__ import annotations

import numpy as np
import torch


def mapping_trace(events: torch.Tensor, stream_offsets: torch.Tensor, num_regions: int, num_pcs: int,
                  execs_per_begin: int = 2):
    """events: uint8 [N * 16] marker records; stream_offsets: int64 [S + 1].
    Returns (events uint8 [N' * 16], stream_offsets int64 [S + 1]) with region ids 0 .. R-1 kept and exec
    records under region id R = num_regions. PCs: every region owns a range of PCs, and the last exec record
    after each begin uses one of eight helper PCs shared by all regions (so their ownership is ambiguous)."""
    dev = events.device
    w = events.view(torch.int64).view(-1, 2)
    n = w.shape[0]
    K = int(execs_per_begin)
    tagctx = w[:, 1]
    tag = tagctx & 0xFFFFFFFF
    is_begin = (tag & 1) == 0
    reps = torch.where(is_begin, 1 + 2 * K, 1)
    ends = torch.cumsum(reps, 0)
    src = torch.repeat_interleave(torch.arange(n, device=dev), reps)
    pos = torch.arange(src.numel(), device=dev) - (ends - reps)[src]     # 0 = the marker itself
    j = (pos - 1) // 2
    half = (pos - 1) % 2
    region = (tag >> 1)[src]
    ctx = ((tagctx >> 32) & 0xFFFFFFFF)[src]
    own = (region * 331 + j * 7 + ctx % 3) % max(num_pcs - 8, 1)
    shared = num_pcs - 1 - (region % 8)
    pc = torch.where(j == K - 1, shared, own) % num_pcs
    count = 1 + (src + j) % 4
    is_exec = pos > 0
    out = torch.empty((src.numel(), 2), dtype=torch.int64, device=dev)
    out[:, 0] = torch.where(is_exec, torch.where(half == 1, count, torch.zeros_like(count)), w[:, 0][src])
    exec_tag = (num_regions << 1) | half
    out[:, 1] = torch.where(is_exec, exec_tag | (pc << 32), tagctx[src])
    new_off = torch.zeros_like(stream_offsets)
    idx = stream_offsets.to(dev) - stream_offsets[0].to(dev)
    nz = idx > 0
    new_off[nz] = ends[idx[nz] - 1]
    return out.view(torch.uint8).reshape(-1), new_off


def decode_mapping_trace(events: np.ndarray, num_regions: int):
    """Encoded marker records (structured array with ts, tag, ctx) -> (kind, id, count) arrays of the abstract
    mapping-run records: 0 begin(region), 1 end(region), 2 exec(pc, count). Assumes every exec pair is intact."""
    region = events["tag"] >> 1
    is_end = (events["tag"] & 1).astype(bool)
    ex = region == num_regions
    keep = ~(ex & is_end)                       # drop the end half of every exec pair
    idx = np.nonzero(keep)[0]
    kind = np.where(ex[idx], 2, is_end[idx].astype(np.int64)).astype(np.uint32)
    ident = np.where(ex[idx], events["ctx"][idx], region[idx]).astype(np.uint32)
    nxt = np.minimum(idx + 1, len(events) - 1)
    count = np.where(ex[idx], events["ts"][nxt], 0).astype(np.uint64)
    removed_before = np.cumsum(~keep)
    return kind, ident, count, removed_before


def encode_map_events(kind: np.ndarray, ident: np.ndarray, count: np.ndarray, exec_region: int) -> np.ndarray:
    """Mapping-run records (kind 0 begin / 1 end of region `ident`, 2 = PC index `ident` executed `count`
    times) in the marker encoding argus.h documents: an exec record becomes a begin/end pair of region
    `exec_region` with ctx = PC index and ts 0 / count. Returns (events, source index of each event).
    Input preparation: the library itself only ever sees marker records."""
    kind = np.asarray(kind)
    is_exec = kind == 2
    reps = np.where(is_exec, 2, 1)
    src = np.repeat(np.arange(len(kind)), reps)
    second = np.zeros(len(src), dtype=bool)
    second[np.cumsum(reps)[is_exec] - 1] = True           # the end half of every exec pair
    ev = np.zeros(len(src), dtype=np.dtype([("ts", "<u8"), ("tag", "<u4"), ("ctx", "<u4")]))
    ex = is_exec[src]
    ev["tag"] = np.where(ex, (exec_region << 1) | second, (np.asarray(ident)[src] << 1) | (kind[src] & 1)).astype(np.uint32)
    ev["ctx"] = np.where(ex, np.asarray(ident)[src], 0).astype(np.uint32)
    ev["ts"] = np.where(second, np.asarray(count)[src], 0).astype(np.uint64)
    return ev, src
