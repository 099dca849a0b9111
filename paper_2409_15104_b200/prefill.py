"""Call sequences over the C ABI for the three ways the path is driven.

Orchestration only (which call, which buffer): all arithmetic happens inside libpec.so.

* PartitionedPrefill  - the per-step work of ring-attention sequence parallelism run as
  virtual partitions on one GPU: plan, one launch per zigzag KV partition, each merging its
  result into the running (O, LSE) state in its epilogue (or, chain=False, one partial per
  partition and n-way LSE merge passes).
* chunked_prefill     - a long prefill cut into preemptible chunks, each resumed from the
  stored K/V prefix (the pause points fall between kernel launches).
* varlen_prefill      - a packed batch of short requests.
* StreamedPrefill     - consecutive partitioned prefills whose inputs come from and whose results go to
  host memory: the copies of neighbouring steps overlap the compute of the current one.
* ring_prefill        - ring-attention sequence parallelism with every rank emulated on one GPU:
  rank r keeps the query rows of its own zigzag segment and meets one K/V segment per ring step.
"""
import torch

from . import binding


class PartitionedPrefill:
    """Buffers and call sequence for P virtual sequence partitions combined through their LSE.

    chain=True (default): one fp32 state; the launch of each partition merges its own result into
    it in the attention epilogue (the online-softmax step across key segments), the last launch
    writing the final output in the input dtype.  Partition 0 goes last because every row sees some
    key of it, so the launch that rounds to the output dtype covers all rows.
    chain=False: partials are kept in up to `max_live` fp32 buffers (bounded by
    `partial_budget_bytes`) and merged with one n-way pass per group instead of P-1 two-way passes;
    with two buffers this degenerates to the running two-way merge.
    """

    def __init__(self, seq_len, hq, num_parts, dtype, device, part_align=128, partial_budget_bytes=80 << 30, chain=True):
        self.S, self.Hq, self.P, self.align = seq_len, hq, num_parts, part_align
        self.dtype = dtype
        self.chain = chain
        f32 = torch.float32
        per_partial = seq_len * hq * (128 * 4 + 4)
        self.max_live = max(2, min(num_parts, binding.PEC_MERGE_MAX_PARTS, partial_budget_bytes // max(per_partial, 1)))
        n_buf = 0 if num_parts == 1 else (1 if chain else self.max_live)
        self.part_o = [torch.empty((seq_len, hq, 128), dtype=f32, device=device) for _ in range(n_buf)]
        self.part_l = [torch.empty((seq_len, hq), dtype=f32, device=device) for _ in range(n_buf)]
        self.out_o = torch.empty((seq_len, hq, 128), dtype=dtype, device=device)
        self.out_l = torch.empty((seq_len, hq), dtype=f32, device=device)
        self.attn_events = []      # (start, end) CUDA events per attention launch when timing
        self.merge_events = []
        self.merge_parts = []      # parts merged by each merge launch of the last run

    def merge_launches(self):
        """Merge launches per step: the first group holds max_live partials, later ones max_live-1 new ones."""
        if self.P == 1 or self.chain:
            return 0
        rest = self.P - self.max_live
        return 1 + (0 if rest <= 0 else -(-rest // (self.max_live - 1)))

    def launches_per_step(self):
        # chain: the first launch (partition 1) also fills the rows below that partition's first key
        return self.P + (1 if self.chain and self.P > 1 else self.merge_launches())

    def run(self, q, k, v, stream=None, time_kernels=False, out=None):
        """Returns (o [S,Hq,128] in the input dtype, lse [S,Hq] fp32); `out` = (o, lse) buffers to write the
        result to instead of the runner's own.  time_kernels=True brackets every launch with CUDA events and, so
        that those mean something, lets no launch start before its predecessor has finished."""
        P = self.P
        out_o, out_l = (self.out_o, self.out_l) if out is None else out
        self.plan = binding.pec_plan_partitions(self.S, P, 0, self.align, 128, 128, True, tiles=False)
        self.merge_parts = []
        if P == 1:
            self._attn(q, k, v, 0, out_o, out_l, stream, time_kernels)
            return out_o, out_l
        if self.chain:
            st_o, st_l = self.part_o[0], self.part_l[0]
            self._attn(q, k, v, 1, st_o, st_l, stream, time_kernels)
            # q, k, v were there before the first launch: every later launch of the chain may start on the SMs its
            # predecessor has left (it waits for that launch before it touches the state)
            for part in range(2, P):
                self._attn(q, k, v, part, st_o, st_l, stream, time_kernels, acc=(st_o, st_l), overlap=not time_kernels)
            self._attn(q, k, v, 0, out_o, out_l, stream, time_kernels, acc=(st_o, st_l), overlap=not time_kernels)
            return out_o, out_l
        p = 0
        first = True
        while p < P:
            # buffer 0 holds the running result after the first group
            slots = list(range(0 if first else 1, self.max_live))
            used = []
            for b in slots:
                if p >= P:
                    break
                self._attn(q, k, v, p, self.part_o[b], self.part_l[b], stream, time_kernels)
                used.append(b)
                p += 1
            group = used if first else [0] + used
            last = p >= P
            ev = self._events(time_kernels, self.merge_events, stream)
            o_parts, l_parts = [self.part_o[b] for b in group], [self.part_l[b] for b in group]
            if len(group) == 2 and not last:
                binding.pec_attn_merge(o_parts[0], l_parts[0], o_parts[1], l_parts[1], inplace=True, stream=stream)
            elif len(group) == 2:
                binding.pec_attn_merge(o_parts[0], l_parts[0], o_parts[1], l_parts[1], o_out=out_o,
                                       lse_out=out_l, stream=stream)
            elif last:
                binding.pec_attn_merge_n(o_parts, l_parts, o_out=out_o, lse_out=out_l, stream=stream)
            else:
                binding.pec_attn_merge_n(o_parts, l_parts, inplace=True, stream=stream)
            if ev:
                ev[1].record(stream)
            self.merge_parts.append(len(group))
            first = False
        return out_o, out_l

    def _events(self, on, store, stream):
        if not on:
            return None
        ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
        ev[0].record(stream)
        store.append(ev)
        return ev

    def _attn(self, q, k, v, p, o, l, stream, time_kernels, acc=None, overlap=False):
        ev = self._events(time_kernels, self.attn_events, stream)
        binding.pec_prefill_attn(q, k, v, seq_len=self.S, part_id=p, num_parts=self.P, part_align=self.align,
                                 causal=True, o=o, lse=l, stream=stream, acc=acc, overlap_previous=overlap)
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


def make_worklist(cu_host, dtype, device):
    """Heaviest-first tile list of a packed batch for the kernel that handles `dtype`, on the device
    (cu_host: host sequence of B + 1 row offsets)."""
    items = binding.pec_plan_worklist(cu_host, binding.pec_worklist_block_m(dtype), 128, True)
    return torch.from_numpy(items).to(device, non_blocking=True)


def varlen_prefill(q, k, v, cu_seqlens, o=None, lse=None, stream=None, worklist=None):
    """Packed batch of short causal prefills (cu_seqlens: int32 CUDA tensor [B+1]; worklist: optional
    tensor from make_worklist - without it every CTA searches cu_seqlens for its tile)."""
    return binding.pec_prefill_attn(q, k, v, cu_seqlens=cu_seqlens, causal=True, o=o, lse=lse, stream=stream,
                                    worklist=worklist)


def ring_prefill(q, k, v, num_parts, part_align=128, stream=None):
    """The P x P (rank, ring step) launches of ring-attention SP (Section 2.2) on one GPU, no rank
    waiting for another: rank r owns the query rows of zigzag partition r and at step t attends to
    the keys of partition (r - t) mod P, one launch per (rank, step) that merges its result into the
    rank's running (O, LSE) state.  Steps run t = 1, ..., P-1, 0: the rank's own keys come last because
    every one of its rows sees some of them, so that launch can round the state to the output dtype.
    Returns (o [S,Hq,128] in the input dtype, lse [S,Hq] fp32, launches)."""
    S, Hq = q.shape[0], q.shape[1]
    P = num_parts
    f32 = torch.float32
    out_o = torch.empty((S, Hq, 128), dtype=q.dtype, device=q.device)
    out_l = torch.empty((S, Hq), dtype=f32, device=q.device)
    if P == 1:
        binding.pec_prefill_attn(q, k, v, seq_len=S, causal=True, o=out_o, lse=out_l, stream=stream)
        return out_o, out_l, 1
    st_o = torch.empty((S, Hq, 128), dtype=f32, device=q.device)    # every rank's state lives in its own rows
    st_l = torch.empty((S, Hq), dtype=f32, device=q.device)
    launches = 0
    for r in range(P):
        order = list(range(1, P)) + [0]
        for i, t in enumerate(order):
            first, last = i == 0, i == P - 1
            # every launch after the very first may overlap its predecessor: the inputs were there before either
            binding.pec_prefill_attn(q, k, v, seq_len=S, part_id=(r - t) % P, num_parts=P, part_align=part_align,
                                     q_part_id=r, q_num_parts=P, causal=True,
                                     o=out_o if last else st_o, lse=out_l if last else st_l,
                                     acc=None if first else (st_o, st_l), stream=stream, overlap_previous=launches > 0)
            launches += 1
    return out_o, out_l, launches


class StreamedPrefill:
    """Host-to-host pipelining of consecutive prefills run by a PartitionedPrefill: while step i computes,
    the inputs of step i+1 are copied to the device and the result of step i-1 is copied back (three
    streams, two sets of device input and output buffers; PCIe carries both directions at once).
    Host tensors must be pinned.  Orchestration only: every copy is a cudaMemcpyAsync issued by torch,
    every computation a call of the library."""

    def __init__(self, runner, hkv, device):
        self.runner = runner
        S, Hq, dt = runner.S, runner.Hq, runner.dtype
        self.inp = [tuple(torch.empty((S, h, 128), dtype=dt, device=device) for h in (Hq, hkv, hkv)) for _ in range(2)]
        self.out = [(torch.empty((S, Hq, 128), dtype=dt, device=device),
                     torch.empty((S, Hq), dtype=torch.float32, device=device)) for _ in range(2)]
        self.s_in, self.s_comp, self.s_out = (torch.cuda.Stream(device=device) for _ in range(3))
        self.computed = [None, None]      # event: the step that last used buffer set b has finished computing
        self.copied_out = [None, None]    # event: its result has left the device
        self.step = 0

    def submit(self, q_h, k_h, v_h, o_h, l_h):
        """Enqueue one prefill: q_h, k_h, v_h -> device -> (o_h, l_h).  Returns at once."""
        b = self.step & 1
        self.step += 1
        with torch.cuda.stream(self.s_in):
            if self.computed[b] is not None:
                self.s_in.wait_event(self.computed[b])           # the inputs of two steps ago are no longer read
            for dst, src in zip(self.inp[b], (q_h, k_h, v_h)):
                dst.copy_(src, non_blocking=True)
            arrived = torch.cuda.Event(); arrived.record(self.s_in)
        with torch.cuda.stream(self.s_comp):
            self.s_comp.wait_event(arrived)
            if self.copied_out[b] is not None:
                self.s_comp.wait_event(self.copied_out[b])       # the result of two steps ago has been read out
            self.runner.run(*self.inp[b], stream=self.s_comp, out=self.out[b])
            self.computed[b] = torch.cuda.Event(); self.computed[b].record(self.s_comp)
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(self.computed[b])
            o_h.copy_(self.out[b][0], non_blocking=True)
            l_h.copy_(self.out[b][1], non_blocking=True)
            self.copied_out[b] = torch.cuda.Event(); self.copied_out[b].record(self.s_out)

    def drain(self):
        for s in (self.s_in, self.s_comp, self.s_out):
            s.synchronize()
