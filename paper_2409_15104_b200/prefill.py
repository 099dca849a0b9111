"""Call sequences over the C ABI for the three ways the path is driven.

Orchestration only (which call, which buffer): all arithmetic happens inside libpec.so.

* partitioned_prefill - the per-step work of ring-attention sequence parallelism run as
  virtual partitions on one GPU: plan, one partial per zigzag KV partition, running LSE merge.
* chunked_prefill     - a long prefill cut into preemptible chunks, each resumed from the
  stored K/V prefix (the pause points fall between kernel launches).
* varlen_prefill      - a packed batch of short requests.
"""
import torch

from . import binding


class PartitionedPrefill:
    """Buffers and call sequence for P virtual sequence partitions merged through their LSE."""

    def __init__(self, seq_len, hq, num_parts, dtype, device, part_align=128):
        self.S, self.Hq, self.P, self.align = seq_len, hq, num_parts, part_align
        self.dtype = dtype
        f32 = torch.float32
        self.acc_o = torch.empty((seq_len, hq, 128), dtype=f32, device=device)
        self.acc_l = torch.empty((seq_len, hq), dtype=f32, device=device)
        if num_parts > 1:
            self.tmp_o = torch.empty_like(self.acc_o)
            self.tmp_l = torch.empty_like(self.acc_l)
        self.out_o = torch.empty((seq_len, hq, 128), dtype=dtype, device=device)
        self.out_l = torch.empty((seq_len, hq), dtype=f32, device=device)
        self.attn_events = []      # (start, end) CUDA events per attention launch when timing
        self.merge_events = []

    def launches_per_step(self):
        return self.P + (self.P - 1) if self.P > 1 else 1

    def run(self, q, k, v, stream=None, time_kernels=False):
        """Returns (o [S,Hq,128] in the input dtype, lse [S,Hq] fp32)."""
        P = self.P
        plan = binding.pec_plan_partitions(self.S, P, 0, self.align, 128, 128, True, tiles=False)
        self.plan = plan
        if P == 1:
            self._attn(q, k, v, 0, self.out_o, self.out_l, stream, time_kernels)
            return self.out_o, self.out_l
        for p in range(P):
            o, l = (self.acc_o, self.acc_l) if p == 0 else (self.tmp_o, self.tmp_l)
            self._attn(q, k, v, p, o, l, stream, time_kernels)
            if p == 0:
                continue
            ev = self._events(time_kernels, self.merge_events, stream)
            if p < P - 1:
                binding.pec_attn_merge(self.acc_o, self.acc_l, o, l, inplace=True, stream=stream)
            else:
                binding.pec_attn_merge(self.acc_o, self.acc_l, o, l, o_out=self.out_o, lse_out=self.out_l,
                                       stream=stream)
            if ev:
                ev[1].record(stream)
        return self.out_o, self.out_l

    def _events(self, on, store, stream):
        if not on:
            return None
        ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
        ev[0].record(stream)
        store.append(ev)
        return ev

    def _attn(self, q, k, v, p, o, l, stream, time_kernels):
        ev = self._events(time_kernels, self.attn_events, stream)
        binding.pec_prefill_attn(q, k, v, seq_len=self.S, part_id=p, num_parts=self.P, part_align=self.align,
                                 causal=True, o=o, lse=l, stream=stream)
        if ev:
            ev[1].record(stream)


def chunked_prefill(q, k, v, chunk_len, o, lse, stream=None, between_chunks=None, events=None):
    """Run a long causal prefill as chunks of `chunk_len` query rows.  Chunk c reads only keys
    [0, end of chunk c).  between_chunks(c) is called on the host after chunk c is enqueued
    (the preemption point: other work may be launched there).  Returns the chunk list."""
    S = q.shape[0]
    plan = binding.pec_plan_partitions(S, 1, chunk_len, 128, 128, 128, True, tiles=False)
    for c, (start, n) in enumerate(plan["chunks"]):
        if events is not None:
            ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
            ev[0].record(stream)
        binding.pec_prefill_attn(q, k, v, seq_len=S, chunk_start=start, chunk_len=n, kv_len=start + n,
                                 causal=True, o=o[start:start + n], lse=lse[start:start + n], stream=stream)
        if events is not None:
            ev[1].record(stream)
            events.append(ev)
        if between_chunks is not None:
            between_chunks(c)
    return plan["chunks"]


def varlen_prefill(q, k, v, cu_seqlens, o=None, lse=None, stream=None):
    """Packed batch of short causal prefills (cu_seqlens: int32 CUDA tensor [B+1])."""
    return binding.pec_prefill_attn(q, k, v, cu_seqlens=cu_seqlens, causal=True, o=o, lse=lse, stream=stream)
