"""Seeded synthetic inputs shaped like the paper's workloads.

Holds no attention arithmetic: only random tensors, request lengths and the five
workload descriptions.  Both the GPU path's tests/benchmarks and the CPU oracle's
callers draw their inputs here so that they see identical bits.

Shapes follow the paper's evaluation set-up (Section 6.2): short inputs follow the
Azure trace's shape (about 80 % of inputs under 2K tokens, maximum near 9K), long
inputs are 100K-500K tokens, and the models use grouped-query attention
(Section 5.3) with Llama-3-class head shapes.  The trace itself is not used: lengths
are drawn from a lognormal with median 700 and P(L < 2048) = 0.80, capped at 8192.
"""
import math
import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field

import numpy as np
import torch

BASE_SEED = 20240915
_CHUNK = 1 << 24  # elements per independently keyed block

LOGN_MU = math.log(700.0)
LOGN_SIGMA = math.log(2048.0 / 700.0) / 0.8416212335729143  # z_{0.80}
MAX_SHORT_LEN = 8192


def normal_tensor(seed: int, stream: int, shape, dtype=torch.bfloat16) -> torch.Tensor:
    """i.i.d. N(0,1) values, rounded (nearest-even) to `dtype`, as a CPU tensor.

    Counter-based: block b of the flattened tensor uses Philox keyed by
    (seed, stream, b), so the result does not depend on how it is consumed.
    """
    n = int(np.prod(shape)) if len(shape) else 1
    out = torch.empty(n, dtype=dtype)

    def fill(b):
        start = b * _CHUNK
        cnt = min(_CHUNK, n - start)
        key = (int(seed) << 20) ^ (int(stream) << 12) ^ b
        gen = np.random.Generator(np.random.Philox(key=key))
        block = gen.standard_normal(cnt, dtype=np.float32)
        out[start:start + cnt] = torch.from_numpy(block).to(dtype)

    n_blocks = (n + _CHUNK - 1) // _CHUNK
    if n_blocks <= 1:
        for b in range(n_blocks):
            fill(b)
    else:
        workers = max(1, min(n_blocks, len(os.sched_getaffinity(0))))
        with ThreadPoolExecutor(workers) as pool:
            list(pool.map(fill, range(n_blocks)))
    return out.reshape(*shape)


def qkv(seed: int, tokens: int, hq: int, hkv: int, d: int = 128, dtype=torch.bfloat16):
    """Q [tokens,hq,d], K and V [tokens,hkv,d] ~ N(0,1), one sub-stream per tensor."""
    q = normal_tensor(seed, 1, (tokens, hq, d), dtype)
    k = normal_tensor(seed, 2, (tokens, hkv, d), dtype)
    v = normal_tensor(seed, 3, (tokens, hkv, d), dtype)
    return q, k, v


def short_lengths(seed: int, batch: int) -> list:
    """Request lengths L = clamp(round(exp(mu + sigma z)), 1, 8192), z ~ N(0,1)."""
    gen = np.random.Generator(np.random.Philox(key=int((seed << 20) ^ (7 << 12))))
    z = gen.standard_normal(batch)
    raw = np.exp(LOGN_MU + LOGN_SIGMA * z)
    return [int(min(MAX_SHORT_LEN, max(1, round(float(x))))) for x in raw]


def cu_seqlens(lengths) -> list:
    out = [0]
    for n in lengths:
        out.append(out[-1] + int(n))
    return out


@dataclass
class Workload:
    name: str
    seed: int
    hq: int
    hkv: int
    dtype: torch.dtype
    seq_len: int = 0            # single long request (0 for pure varlen batches)
    num_parts: int = 1          # zigzag sequence partitions merged through LSE
    chunk_len: int = 0          # >0: preemptible chunks of this many query rows
    short_batch: int = 0        # >0: colocated / stand-alone varlen batch size
    d: int = 128
    part_align: int = 128
    note: str = ""
    extra: dict = field(default_factory=dict)


WORKLOADS = {
    "c1": Workload("c1", BASE_SEED + 1, 8, 8, torch.float32, seq_len=1024, num_parts=4,
                   note="S=1024 fp32, 4 zigzag partitions merged via LSE"),
    "c2": Workload("c2", BASE_SEED + 2, 32, 8, torch.bfloat16, short_batch=64,
                   note="64 short requests, lognormal lengths, varlen-packed"),
    "c3": Workload("c3", BASE_SEED + 3, 32, 8, torch.bfloat16, seq_len=32768, num_parts=8,
                   note="S=32768, 8 zigzag partitions merged on device"),
    "c4": Workload("c4", BASE_SEED + 4, 32, 8, torch.bfloat16, seq_len=131072, chunk_len=8192,
                   short_batch=32,
                   note="S=131072 as 16 resumed chunks + colocated 32-request varlen batch"),
    "c5": Workload("c5", BASE_SEED + 5, 64, 8, torch.bfloat16, seq_len=262144, num_parts=16,
                   note="S=262144, 64/8 heads, 16 zigzag partitions merged on device"),
}


def causal_pairs(seq_len: int) -> int:
    """Visible (query, key) pairs per head of one causal request."""
    return seq_len * (seq_len + 1) // 2


def attention_flops(pairs_per_head: int, hq: int, d: int = 128) -> int:
    """2 multiply-adds per pair per channel for QK^T and again for PV."""
    return 4 * d * hq * pairs_per_head
