"""Benchmark of the prefix-hit path on B200.

A step is one pass of the whole path over one batch of synthetic prompts:
    lookup_fetch(PIN) -> reserve(room for the batch's new blocks) -> insert -> release
on the Llama-3-8B KV shape (32 layers x 8 KV heads x 128, bf16, 16-token blocks), a 20,000-block store
pool in HBM, 500 documents of 2k-6k tokens with Zipf(1.1) popularity, 64 prompts per batch, each a
document plus a unique 64-256-token question.  No call waits for the host: matched lengths, free counts and
the number of victims stay on the device.

Prints ONE JSON line.  `value` is the KV bytes DRAM has to move for the fetches and inserts of the timed steps
(each distinct source block read once, every delivered or stored block written once, stored blocks read once)
divided by the time of the whole steps, inputs resident in HBM; `value_delivered_bytes` counts 2 x block bytes
per delivered block instead.  `e2e` repeats the measurement with the step's token ids / offsets / block tables
copied from pinned host memory and its results copied back inside the timed region.  `roofline` is the fetch
copy kernel alone (events recorded around that kernel by the library) against the measured HBM copy bandwidth.
`latency` holds small-batch steps (1 / 4 / 16 prompts of 4k tokens that hit), `lookup` the 10^6-node lookup
stress, `cpu_baseline` the CPU oracle timed on this machine on a bounded sample of the same stream.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload ...] ...
With --gpus N > 1 (or under torchrun) every rank runs an independent replica on its own GPU (the path has no
exchange step); rank 0 prints the aggregate.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2607_22648_b200 import workloads as W  # noqa: E402

NOMINAL_HBM_GBS = 8000.0
# DRAM bytes of the fetch copy kernel per block, from the ncu capture of a small case (profiles/): traffic grows in
# proportion to the blocks read and written, so a full launch is MODELLED as these factors times its block counts.
NCU_READ_FACTOR = 1.00    # dram__bytes_read.sum / (distinct source blocks x block bytes)
NCU_WRITE_FACTOR = 0.99   # dram__bytes_write.sum / (delivered blocks x block bytes)
FALLBACK_HBM_GBS = 6650.0
# L2 read sectors per issued probe of lookup_kernel on the 10^6-node stress, from the ncu capture in profiles/
L2_SECTORS_PER_PROBE = 8.3


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Polls SM clock and clock-event reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index, period=0.01):
        self.index, self.period, self.rows, self.stop_flag, self.t = index, period, [], False, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
        except Exception:
            self.nv = None

    def start(self):
        if self.nv is None:
            return
        self.stop_flag = False
        self.rows = []
        self.t = threading.Thread(target=self._poll, daemon=True)
        self.t.start()

    def _poll(self):
        nv = self.nv
        while not self.stop_flag:
            try:
                clk = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    rs = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    rs = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.rows.append((clk, rs))
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        if self.nv is None or self.t is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvml unavailable"], "samples": 0}
        self.stop_flag = True
        self.t.join(timeout=2)
        nv = self.nv
        try:
            mx = float(nv.nvmlDeviceGetMaxClockInfo(self.h, nv.NVML_CLOCK_SM))
        except Exception:
            mx = None
        bits = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4,
                "hw_power_brake": 0x80}
        reasons = set()
        for _, rs in self.rows:
            for name, bit in bits.items():
                if rs & bit:
                    reasons.add(name)
        clk = [c for c, _ in self.rows]
        return {"sm_mhz": float(np.median(clk)) if clk else None, "sm_max_mhz": mx, "reasons": sorted(reasons), "samples": len(clk)}


# ---------------------------------------------------------------------------------------------------------
class Serving:
    """Serving-loop workloads: llama8b = configs[1] (the one the metric is quoted on), llama70b = configs[3],
    churn = configs[4] (HBM + pinned-host tiers)."""

    def __init__(self, args, rank, kind="llama8b"):
        import torch
        from paper_2607_22648_b200 import binding as G
        self.torch, self.G, self.kind = torch, G, kind
        free_gb = torch.cuda.mem_get_info()[0] / 1e9
        host_blocks = 0
        if kind == "llama8b":
            bt = args.block_tokens or 16
            self.sh = W.KVShape(32, 8, 128, bt)
            self.batch, self.pool_blocks = args.batch or 64, args.pool_blocks or 20000 * 16 // bt
            self.stream = W.llama8b_stream(seed=W.BASE_SEED + 1 + 1000 * rank, n_docs=args.docs or 500, shape=self.sh)
            self.name = "llama3_8b_kv_pool%dk_zipf1.1_batch%d" % (self.pool_blocks // 1000, self.batch) if bt == 16 else \
                "llama3_8b_kv_block%d_pool%d_zipf1.1_batch%d" % (bt, self.pool_blocks, self.batch)
            self.kv = "32L x 8H x 128 bf16, block %d" % bt
        elif kind == "multiturn":
            self.sh = W.LLAMA3_8B
            self.batch, self.pool_blocks = args.batch or 64, args.pool_blocks or 20000
            self.stream = W.conversation_stream(seed=W.BASE_SEED + 5 + 1000 * rank, n_conversations=args.docs or 512)
            self.name = "multiturn_llama3_8b_kv_pool%d_conv%d_batch%d" % (self.pool_blocks, self.stream.n_conversations, self.batch)
            self.kv = "32L x 8H x 128 bf16, block 16"
        elif kind == "llama70b":
            self.sh = W.LLAMA3_70B
            self.batch = args.batch or 8
            self.stream = W.llama70b_stream(seed=W.BASE_SEED + 3 + 1000 * rank, n_docs=args.docs or 18)
            cache_gb = self.batch * self.stream.max_blocks * self.sh.block_bytes / 1e9
            self.pool_blocks = args.pool_blocks or int(min(9536, (free_gb - cache_gb - 8) * 1e9 // self.sh.block_bytes))
            self.name = "llama3_70b_kv_pool%d_zipf1.2_batch%d_16k_prefix" % (self.pool_blocks, self.batch)
            self.kv = "80L x 8H x 128 bf16, block 32"
        else:
            self.sh = W.LLAMA3_8B
            self.batch, self.pool_blocks = args.batch or 16, args.pool_blocks or 19073
            self.stream = W.churn_stream(seed=W.BASE_SEED + 4 + 1000 * rank, n_docs=args.docs or 5000)
            host_gb = args.host_gb if args.host_gb else pinnable_host_gb()
            host_blocks = int(host_gb * 1e9 // self.sh.block_bytes)
            self.name = "churn_llama3_8b_kv_hbm%d_host%d_zipf1.0_batch%d" % (self.pool_blocks, host_blocks, self.batch)
            self.kv = "32L x 8H x 128 bf16, block 16"
        self.host_blocks = host_blocks
        self.promote = args.promote if host_blocks else 0
        self.async_demote = bool(args.async_demote and host_blocks)
        self.mb = self.stream.max_blocks
        flags = (G.COPY_BULK if args.engine == "bulk" else G.COPY_VECTOR) | G.copy_variant(args.variant) | \
            G.copy_ctas_per_sm(args.ctas_per_sm) | (G.EVICT_GDSF if args.policy == "gdsf" else 0)
        self.store = G.PTStore(self.sh.layers, self.sh.heads, self.sh.dim, self.sh.block_tokens, self.pool_blocks,
                               max_requests=self.batch, max_batch_blocks=self.batch * self.mb, flags=flags, host_blocks=host_blocks)
        self.rng = np.random.default_rng(W.BASE_SEED + 77 + rank)
        self.steps = []
        self.cache = None

    def prepare(self, n_steps):
        """Generate every batch up front (host + device copies) and size the paged cache for the largest."""
        torch = self.torch
        B = self.sh.block_tokens
        raw, need_max = [], 0
        for _ in range(n_steps):
            seqs, _tags = self.stream.batch(self.batch)
            need = sum(len(s) // B for s in seqs)
            need_max = max(need_max, need)
            raw.append((seqs, need))
        self.cache_blocks = need_max + 16
        self.cache = self.G.PagedKV(self.sh.layers, self.cache_blocks, self.sh.chunk_bytes)
        noise = torch.randint(0, 256, (2, 61, self.sh.chunk_bytes), dtype=torch.uint8, device="cuda")
        pick = torch.arange(self.cache_blocks, device="cuda") % 61
        for t in self.cache.tensors:                       # any bytes will do for timing; make them non-trivial
            torch.index_select(noise, 1, pick, out=t)
        for seqs, need in raw:
            toks, offs = W.ragged(seqs)
            bt = W.shuffled_block_tables(self.rng, seqs, B, self.mb, self.cache_blocks)
            nblk = np.array([len(s) // B for s in seqs], dtype=np.int64)
            host = dict(tokens=torch.from_numpy(toks).pin_memory(), offsets=torch.from_numpy(offs).pin_memory(),
                        bt=torch.from_numpy(bt).pin_memory())
            devc = {k: v.cuda() for k, v in host.items()}
            self.steps.append(dict(host=host, dev=devc, nblk=nblk, total_blocks=int(nblk.sum())))
        R = self.batch
        self.matched = torch.empty(R, dtype=torch.int32, device="cuda")
        self.ids = torch.empty((R, self.mb), dtype=torch.int32, device="cuda")
        self.ins_ids = torch.empty((R, self.mb), dtype=torch.int32, device="cuda")
        self.newb = torch.empty(R, dtype=torch.int32, device="cuda")
        self.nev = torch.zeros(2, dtype=torch.int32, device="cuda")
        self.nprom = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.h_matched = torch.empty(R, dtype=torch.int32).pin_memory()
        self.h_ids = torch.empty((R, self.mb), dtype=torch.int32).pin_memory()
        self.h_newb = torch.empty(R, dtype=torch.int32).pin_memory()

    def step(self, i, e2e=False, events=None):
        """One pass of the path.  Returns nothing; counters come from ptstore_stats.  No host synchronisation inside."""
        torch, G, st = self.torch, self.G, self.store
        s = self.steps[i]
        if e2e:
            d = {k: v.to("cuda", non_blocking=True) for k, v in s["host"].items()}
        else:
            d = s["dev"]
        want = s["total_blocks"] + self.promote              # free HBM blocks the insert needs (+ room for the next promotions)
        timed = events is not None
        if self.promote or self.async_demote:                # promotion sits between lookup and fetch; an asynchronous
            st.lookup(d["tokens"], d["offsets"], self.mb, G.PIN, self.matched, self.ids)     # demotion starts before the fetch
            if self.promote:
                a = self._ev() if timed else None
                st.promote(self.ids, self.matched, G.PINNED_LIST, self.promote, self.nprom)
                if timed:
                    events["promote"].append((a, self._ev()))
            if self.async_demote:
                self._reserve(want, G.ASYNC_COPY, events)    # its copy (device -> host) overlaps the fetch (host -> device)
            a = self._ev() if timed else None
            if timed:
                self._time_copy(events["fetch_copy"])
            st.fetch(self.ids, self.matched, self.cache, d["bt"])
            if timed:
                events["fetch"].append((a, self._ev()))
            if not self.async_demote:
                self._reserve(want, 0, events)
        else:
            a = self._ev() if timed else None
            if timed:
                self._time_copy(events["fetch_copy"])
            st.lookup_fetch(d["tokens"], d["offsets"], self.mb, self.cache, d["bt"], G.PIN, self.matched, self.ids)
            if timed:
                events["fetch"].append((a, self._ev()))
            self._reserve(want, 0, events)
        a = self._ev() if timed else None
        if timed:
            self._time_copy(events["insert_copy"])
        st.insert(d["tokens"], d["offsets"], self.mb, self.cache, d["bt"], self.ins_ids, self.newb, after_lookup=True)
        if timed:
            events["insert"].append((a, self._ev()))
        st.release(self.ids, self.matched)
        if e2e:
            self.h_matched.copy_(self.matched, non_blocking=True)
            self.h_ids.copy_(self.ids, non_blocking=True)
            self.h_newb.copy_(self.newb, non_blocking=True)

    def _reserve(self, want, flags, events):
        a = self._ev() if events is not None else None
        self.store.reserve(want, self.matched, flags, n_evicted=self.nev)
        if events is not None:
            events["evict"].append((a, self._ev()))

    def _time_copy(self, sink):
        """Have the library record two events around the next HBM copy kernel."""
        a, b = self._ev(), self._ev()
        self.store.time_next_copy(a, b)
        sink.append((a, b))

    def _ev(self):
        e = self.torch.cuda.Event(enable_timing=True)
        e.record()
        return e

    def io_bytes(self, i):
        s = self.steps[i]
        h2d = sum(v.numel() * v.element_size() for v in s["host"].values())
        d2h = self.h_matched.numel() * 4 + self.h_ids.numel() * 4 + self.h_newb.numel() * 4
        return h2d, d2h


def reduce_over_ranks(dist, x, op, device):
    """max or sum of a python number over all ranks (identity without a process group)."""
    if dist is None:
        return float(x)
    import torch
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX if op == "max" else dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_throughput(dist, ms, nbytes, device):
    """Replicas: the job's time is the slowest rank's, its work the sum over ranks.  -> (ms, bytes, GB/s)"""
    ms_all = reduce_over_ranks(dist, ms, "max", device)
    bytes_all = reduce_over_ranks(dist, nbytes, "sum", device)
    return ms_all, bytes_all, bytes_all / (ms_all * 1e-3) / 1e9


def init_ranks(backend):
    """(rank, world, local rank, dist or None) from the launcher's environment; one process per GPU."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch
        import torch.distributed as dist
        if backend == "nccl":
            if local >= torch.cuda.device_count():
                raise SystemExit("rank %d has no GPU: %d ranks on %d visible devices" % (rank, world, torch.cuda.device_count()))
            torch.cuda.set_device(local)
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        else:
            dist.init_process_group("gloo")
    return rank, world, local, dist


def relaunch_as_replicas(args):
    """`--gpus N` outside a launcher: start N ranks of this script, one per GPU, and let them report."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=%d" % args.gpus, "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    sys.stdout.flush()
    os.execv(sys.executable, cmd)


def run_stub_replicas(args):
    """The replica launch and aggregation path without a GPU (gloo): every rank pretends to have run K steps and the
    job's figure is combined as for real replicas.  Exercised by the CPU tests."""
    rank, world, local, dist = init_ranks("gloo")
    K = args.steps
    ms = 10.0 + 2.5 * rank                                # the slowest rank sets the job's time
    nbytes = 4.0e9 * K
    if dist:
        dist.barrier()
    ms_all, bytes_all, value = whole_job_throughput(dist, ms, nbytes, "cpu")
    if rank == 0:
        print(json.dumps({"metric": "prefix-hit KV fetch GB/s", "value": round(value, 1), "unit": "GB/s", "n_gpus": world, "steps": K,
                          "warmup": args.warmup, "ms_per_step": round(ms_all / max(K, 1), 4), "higher_is_better": True, "scaling": "weak",
                          "vs_baseline": None, "dtype": "u8", "data": "stub", "config": {"workload": "cpu_stub", "replicas": world}}), flush=True)
    if dist:
        dist.barrier()
        dist.destroy_process_group()


def run_gpu(args):
    import torch
    rank, world, local, dist = init_ranks("nccl")
    if world == 1:
        torch.cuda.set_device(0)
    from __graft_entry__ import build
    if rank == 0:
        build()
    if dist:
        dist.barrier()

    wl = Serving(args, rank, args.workload)
    n_fill, W_, K = args.fill, args.warmup, args.steps
    total_steps = n_fill + W_ + K + (W_ + K if not args.no_e2e else 0)
    wl.prepare(total_steps)
    block_rw = 2 * wl.sh.block_bytes

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(first, count, e2e, events=None):
        s0 = wl.store.stats()
        l0 = wl.store.launch_count()
        barrier()
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        for i in range(first, first + count):
            wl.step(i, e2e=e2e, events=events)
        t1.record()
        barrier()
        ms = t0.elapsed_time(t1)
        s1 = wl.store.stats()
        fetched = (s1.blocks_fetched[0] - s0.blocks_fetched[0]) + (s1.blocks_fetched[1] - s0.blocks_fetched[1])
        distinct = s1.blocks_fetched_distinct - s0.blocks_fetched_distinct
        inserted, demoted, promoted = s1.blocks_inserted - s0.blocks_inserted, s1.blocks_demoted - s0.blocks_demoted, \
            s1.blocks_promoted - s0.blocks_promoted
        moved = fetched + inserted + demoted + promoted
        return dict(ms=ms, fetched=fetched, fetched_host=s1.blocks_fetched[1] - s0.blocks_fetched[1],
                    inserted=inserted, demoted=demoted, host_dropped=s1.blocks_dropped[1] - s0.blocks_dropped[1], promoted=promoted,
                    distinct=distinct, bytes=moved * block_rw, dram_bytes=(distinct + fetched + 2 * (inserted + demoted + promoted)) * wl.sh.block_bytes,
                    launches=wl.store.launch_count() - l0,
                    probes=s1.probes_issued - s0.probes_issued, qblocks=s1.query_blocks - s0.query_blocks,
                    matched=s1.blocks_matched - s0.blocks_matched, dropped=s1.blocks_dropped[0] - s0.blocks_dropped[0])

    i = 0
    for _ in range(n_fill + W_):
        wl.step(i); i += 1
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    events = {"fetch": [], "insert": [], "evict": [], "promote": [], "fetch_copy": [], "insert_copy": []}
    main = timed(i, K, False, events)
    clocks = sampler.stop() if rank == 0 else None
    i += K
    torch.cuda.synchronize()
    ev_ms = {k: sum(a.elapsed_time(b) for a, b in v) for k, v in events.items()}
    fetch_ms, insert_ms, evict_ms, promote_ms = ev_ms["fetch"], ev_ms["insert"], ev_ms["evict"], ev_ms["promote"]
    status = wl.store.status()

    e2e = None
    if not args.no_e2e:
        for _ in range(W_):
            wl.step(i, e2e=True); i += 1
        e2e = timed(i, K, True)
        h2d = int(np.mean([wl.io_bytes(j)[0] for j in range(i, i + K)])); d2h = wl.io_bytes(i)[1]
        i += K

    # aggregate over ranks: max time, sum of bytes
    def agg(x, op):
        return reduce_over_ranks(dist, x, op, "cuda")

    MAX, SUM = "max", "sum"
    ms, total_dram, value = whole_job_throughput(dist, main["ms"], main["dram_bytes"], "cuda")
    delivered_all = agg(main["bytes"], SUM)
    peak, peak_kind = measured_peak()
    host_tier_fetch = bool(wl.host_blocks) or args.engine == "vector"
    # the fetch copy kernel alone: bytes DRAM must move for it / its own duration
    # (with a host tier the fetch is two kernels, one per source tier: the call is timed instead)
    kern_ms = ev_ms["fetch_copy"] if ev_ms["fetch_copy"] > 0 and not wl.host_blocks else fetch_ms
    fetch_dram = (main["distinct"] + main["fetched"]) * wl.sh.block_bytes
    ach = fetch_dram / (kern_ms * 1e-3) / 1e9 if kern_ms > 0 else 0.0
    ach_delivered = main["fetched"] * block_rw / (kern_ms * 1e-3) / 1e9 if kern_ms > 0 else 0.0
    ins_kern_ms = ev_ms["insert_copy"]
    out = {
        "metric": "prefix-hit KV fetch GB/s", "value": round(value, 1), "unit": "GB/s", "n_gpus": world, "steps": K, "warmup": W_,
        "ms_per_step": round(ms / K, 4), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u8", "data": "synthetic",
        "config": {"workload": wl.name, "kv_shape": wl.kv, "pool_blocks": wl.pool_blocks, "host_blocks": wl.host_blocks, "docs": len(getattr(wl.stream, "docs", ())) or wl.stream.n_conversations,
                   "batch": wl.batch, "eviction": args.policy, "engine": args.engine, "variant": args.variant, "l2": "inputs larger than L2 (>= 20 GB per step)",
                   "step": "lookup_fetch(PIN)+reserve+insert_after_lookup+release" if not (wl.promote or wl.async_demote) else "lookup(PIN)+promote+fetch+reserve+insert+release",
                   "fill_steps": n_fill, "replicas": world},
        "value_kind": "bytes DRAM must move (distinct source blocks read once + delivered blocks written + 2 x stored blocks) / step time",
        "frac_of_nominal_8TBps": round(value / world / NOMINAL_HBM_GBS, 4),
        # the same steps counting 2 x block bytes per delivered or stored block (one read and one write each)
        "value_delivered_bytes": round(delivered_all / (ms * 1e-3) / 1e9, 1),
        "per_step": {"blocks_fetched": main["fetched"] / K, "blocks_fetched_distinct": main["distinct"] / K, "blocks_inserted": main["inserted"] / K,
                     "blocks_dropped": main["dropped"] / K,
                     "hit_rate_blocks": round(main["matched"] / max(main["qblocks"], 1), 4),
                     "fetch_call_ms": round(fetch_ms / K, 4), "fetch_copy_kernel_ms": round(ev_ms["fetch_copy"] / K, 4),
                     "insert_call_ms": round(insert_ms / K, 4), "insert_copy_kernel_ms": round(ins_kern_ms / K, 4),
                     "insert_copy_gbps": round(main["inserted"] * block_rw / max(ins_kern_ms, 1e-9) / 1e6, 1),
                     "insert_call_gbps": round(main["inserted"] * block_rw / max(insert_ms, 1e-9) / 1e6, 1),
                     "lookup_probes": main["probes"] / K, "blocks_fetched_from_host": main["fetched_host"] / K,
                     "blocks_demoted": main["demoted"] / K, "host_blocks_dropped": main["host_dropped"] / K,
                     "evict_call_ms": round(evict_ms / K, 4), "blocks_promoted": main["promoted"] / K,
                     "promote_call_ms": round(promote_ms / K, 4),
                     "demote_gbps_one_way": round(main["demoted"] * wl.sh.block_bytes / max(evict_ms, 1e-9) / 1e6, 1),
                     "launches": main["launches"] / K},
        "gpu_launches": int(main["launches"]),
        "device_status": status,
        "clocks": clocks,
        "roofline": {"bound": "hbm", "kernel": "%s (gather of ptstore_lookup_fetch)" % ("copy_vector_kernel<FETCH_MULTI>" if host_tier_fetch else "copy_bulk_multi_kernel"),
                     "achieved": round(ach, 1), "peak": peak, "unit": "GB/s", "frac": round(ach / peak, 4),
                     "peak_kind": peak_kind + " (plain copy, read+write)",
                     "achieved_kind": "bytes DRAM must move per launch (distinct source blocks read once + delivered blocks written) / kernel duration "
                                      "(events recorded around the kernel by the library)",
                     "frac_of_nominal_8TBps": round(ach / NOMINAL_HBM_GBS, 4),
                     "kernel_ms": round(kern_ms / K, 4),
                     "dram_bytes_needed_per_launch": fetch_dram / K,
                     "distinct_source_blocks_per_launch": main["distinct"] / K, "delivered_blocks_per_launch": main["fetched"] / K,
                     "traffic": args.traffic if args.traffic else round(
                         (NCU_READ_FACTOR * main["distinct"] + NCU_WRITE_FACTOR * main["fetched"]) * wl.sh.block_bytes / K),
                     "traffic_kind": "modelled from the small-case ncu capture (profiles/): DRAM bytes per distinct block read and per block "
                                     "written there, times this launch's distinct source blocks and delivered blocks",
                     # counting 2 x block bytes per delivered block; above the copy peak because shared sources are read once
                     "achieved_delivered_bytes": round(ach_delivered, 1), "frac_delivered_bytes": round(ach_delivered / peak, 4)},
    }
    if e2e:
        ems = agg(e2e["ms"], MAX)
        eb = agg(e2e["dram_bytes"], SUM)
        if wl.host_blocks:
            out["host_link_gbps_measured"] = host_link_gbps(torch)
        out["e2e"] = {"value": round(eb / (ems * 1e-3) / 1e9, 1), "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                      "ms_per_step": round(ems / K, 4), "launches_per_step": e2e["launches"] / K}
    if world == 1 and rank == 0:
        # free the serving store before the side records allocate theirs
        wl.store.close()
        wl.cache = None
        wl.store = None
        del wl
        import gc
        gc.collect()
        torch.cuda.empty_cache()
        if not args.no_latency and args.workload == "llama8b":
            out["latency"] = latency_record(args, torch)
            torch.cuda.empty_cache()
        if not args.no_ceilings and args.workload == "llama8b":
            ratio = main["fetched"] / max(main["distinct"], 1)
            ceil = ceilings_record(torch, writes_x100=int(round(ratio * 100)))
            out["copy_engine_ceilings"] = ceil
            mix = [v for k, v in ceil.items() if k.startswith("mix_")][0]
            # the same fraction against what the copy ring itself reaches, live, for a 1:1 copy and for this launch's mix
            # loads and stores measured apart, combined for this launch's byte counts: time = read bytes / read ceiling + written
            # bytes / write ceiling (the memory serves one direction at a time)
            rd, wr = ceil["read_only_4_stages"], ceil["write_only"]
            harmonic = (1 + ratio) / (1 / rd + ratio / wr)
            out["roofline"]["engine_ceilings"] = {"copy_1to1": ceil["copy_1to1"], "mix_of_this_fetch": mix, "writes_per_read": round(ratio, 2),
                                                  "reads_alone": rd, "writes_alone": wr, "reads_and_writes_in_turn": round(harmonic, 1),
                                                  "frac_of_copy_1to1": round(ach / ceil["copy_1to1"], 4), "frac_of_mix": round(ach / mix, 4),
                                                  "frac_of_reads_and_writes_in_turn": round(ach / harmonic, 4),
                                                  "kind": "ptstore_copy_probe in this run (the bulk ring over plain buffers)"}
            torch.cuda.empty_cache()
        if not args.no_lookup and args.workload == "llama8b":
            out["lookup"] = lookup_record(args, torch, K=args.lookup_calls, W_=5)["summary"]
            torch.cuda.empty_cache()
        if not args.no_cpu:
            out["cpu_baseline"] = cpu_oracle_sample(args)
            out["cpu_baseline_all_threads"] = cpu_oracle_threads_sample(args)
    if rank == 0:
        print(json.dumps(out), flush=True)
    if dist:
        dist.barrier()
        dist.destroy_process_group()


def pinnable_host_gb(fraction=0.4, cap=200.0):
    """Budget for the pinned host pool: a fraction of the available RAM, never above the cgroup limit."""
    import psutil
    avail = psutil.virtual_memory().available / 1e9
    for path in ("/sys/fs/cgroup/memory.max", "/sys/fs/cgroup/memory/memory.limit_in_bytes"):
        try:
            lim = open(path).read().strip()
            if lim != "max":
                avail = min(avail, int(lim) / 1e9)
        except Exception:
            pass
    return max(1.0, min(cap, avail * fraction))


def host_link_gbps(torch, gib=1):
    """Pinned-memory cudaMemcpy bandwidth of this machine, both directions (GB/s), best of 3."""
    n = gib << 30
    h = torch.empty(n, dtype=torch.uint8).pin_memory()
    d = torch.empty(n, dtype=torch.uint8, device="cuda")
    out = {}
    for name, (dst, src) in {"h2d": (d, h), "d2h": (h, d)}.items():
        best = 0.0
        for _ in range(3):
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record(); dst.copy_(src, non_blocking=True); b.record(); torch.cuda.synchronize()
            best = max(best, n / (a.elapsed_time(b) * 1e-3) / 1e9)
        out[name] = round(best, 1)
    return out


# ---------------------------------------------------------------------------------------------------------
def latency_record(args, torch, batches=(1, 4, 16), n_docs=32, doc_tokens=4096, suffix_tokens=64, iters=40, headroom=64):
    """Small batches, where the path is latency bound (the paper's end-to-end figure is the time to first token of one
    request): every prompt is a stored 4k-token document (a full hit, 256 blocks = 512 MiB of KV) plus a fresh 64-token
    question (4 new blocks), documents taken round robin so that no two prompts of a batch share one.  A step is
    lookup_fetch(PIN) -> reserve -> insert_after_lookup -> release; the pool has little slack, so room has to be made all the time; a
    reserve that must evict takes `headroom` blocks more than it needs, so most steps find room and skip the eviction.
    Reported per batch size: microseconds of the whole step on the device (steps back to back, calls pre-marshalled), of a
    step seen from the host (first call to the end of a synchronize), of each call, kernel launches per step, and the time
    the step's copies would take at the measured copy bandwidth."""
    import ctypes as C
    from paper_2607_22648_b200 import binding as G
    sh = W.LLAMA3_8B
    B = sh.block_tokens
    doc_blocks, suf_blocks = doc_tokens // B, suffix_tokens // B
    mb = doc_blocks + suf_blocks
    pool = n_docs * doc_blocks + 8 * n_docs * suf_blocks          # slack: suffixes of two rounds over the documents
    bmax = max(batches)
    st = G.PTStore(sh.layers, sh.heads, sh.dim, B, pool, max_requests=bmax, max_batch_blocks=bmax * mb)
    cache = G.PagedKV(sh.layers, bmax * mb, sh.chunk_bytes)
    rng = np.random.default_rng(W.BASE_SEED + 9)
    docs = [rng.integers(0, 128256, size=doc_tokens, dtype=np.int32) for _ in range(n_docs)]

    def dev(a):
        return torch.from_numpy(np.ascontiguousarray(a)).cuda()

    for t in cache.tensors:
        t.random_(0, 256)
    for k in range(0, n_docs, bmax):                                    # store the documents
        part = docs[k:k + bmax]
        toks, offs = W.ragged(part)
        bt = np.arange(len(part) * mb, dtype=np.int32).reshape(len(part), mb)
        st.insert(dev(toks), dev(offs), mb, cache, dev(bt))
    assert st.status() == 0
    peak, _ = measured_peak()
    stream = torch.cuda.current_stream().cuda_stream
    lib, h = G.lib, st.h
    res = {}
    next_doc = 0
    for b in batches:
        n_steps = 8 + 2 * iters
        steps = []
        for _ in range(n_steps):                                        # every step's inputs, resident on the device
            seqs = []
            for _r in range(b):
                seqs.append(np.concatenate([docs[next_doc % n_docs], rng.integers(0, 128256, size=suffix_tokens, dtype=np.int32)]))
                next_doc += 1
            toks, offs = W.ragged(seqs)
            bt = rng.permutation(b * mb).astype(np.int32).reshape(b, mb)
            steps.append((dev(toks), dev(offs), dev(bt)))
        matched = torch.empty(b, dtype=torch.int32, device="cuda")
        ids = torch.empty((b, mb), dtype=torch.int32, device="cuda")
        ins_ids = torch.empty((b, mb), dtype=torch.int32, device="cuda")
        newb = torch.empty(b, dtype=torch.int32, device="cuda")
        nev = torch.zeros(2, dtype=torch.int32, device="cuda")
        cdesc = C.byref(cache.desc)

        def calls(k):
            t, o, bt = steps[k]
            return [
                ("lookup_fetch", lib.ptstore_lookup_fetch, (h, t.data_ptr(), o.data_ptr(), b, mb, G.PIN, cdesc, bt.data_ptr(), matched.data_ptr(), ids.data_ptr(), stream)),
                ("reserve", lib.ptstore_reserve, (h, b * mb, headroom, matched.data_ptr(), b, 0, nev.data_ptr(), None, 0, stream)),
                ("insert", lib.ptstore_insert_after_lookup, (h, t.data_ptr(), o.data_ptr(), b, mb, cdesc, bt.data_ptr(), ins_ids.data_ptr(), newb.data_ptr(), stream)),
                ("release", lib.ptstore_release, (h, ids.data_ptr(), matched.data_ptr(), b, mb, stream)),
            ]

        k = 0
        for _ in range(8):                                              # warm-up
            for _n, f, a in calls(k):
                assert f(*a) == 0
            k += 1
        torch.cuda.synchronize()
        s0, l0 = st.stats(), st.launch_count()
        # (a) steps back to back between two events
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            for _n, f, a in calls(k):
                f(*a)
            k += 1
        e1.record(); torch.cuda.synchronize()
        step_us = e0.elapsed_time(e1) / iters * 1e3
        s1, l1 = st.stats(), st.launch_count()
        # (b) one step at a time: per-call device time and the host's view (first call to end of synchronize)
        per_call = {}
        wall = []
        for _ in range(iters):
            evs = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for q, (_n, f, a) in enumerate(calls(k)):
                evs[q].record(); f(*a)
            evs[4].record()
            torch.cuda.synchronize()
            wall.append((time.perf_counter() - t0) * 1e6)
            for q, (n, _f, _a) in enumerate(calls(k)):
                per_call.setdefault(n, []).append(evs[q].elapsed_time(evs[q + 1]) * 1e3)
            k += 1
        fetched = (s1.blocks_fetched[0] - s0.blocks_fetched[0]) / iters
        inserted = (s1.blocks_inserted - s0.blocks_inserted) / iters
        dropped = (s1.blocks_dropped[0] - s0.blocks_dropped[0]) / iters
        copy_bytes = (fetched + inserted) * 2 * sh.block_bytes
        bound_us = copy_bytes / (peak * 1e9) * 1e6
        res["batch%d" % b] = {"step_us": round(step_us, 1), "step_wall_us": round(float(np.median(wall)), 1),
                              "call_us": {n: round(float(np.median(v)), 1) for n, v in per_call.items()},
                              "launches_per_step": (l1 - l0) / iters, "blocks_fetched": fetched, "blocks_inserted": inserted,
                              "blocks_evicted": dropped, "copy_bytes": copy_bytes, "copy_bound_us": round(bound_us, 1),
                              "step_over_copy_bound": round(step_us / bound_us, 3), "gbps": round(copy_bytes / step_us / 1e3, 1)}
        status = st.status()
        assert status == 0, "status word 0x%x after the batch-%d steps" % (status, b)
    if bmax >= 16:
        res["lookup_fetch_cases"] = lookup_fetch_cases(torch, st, cache, docs, rng, mb, suffix_tokens, peak, sh)
    res["config"] = {"kv_shape": "32L x 8H x 128 bf16, block 16", "prompt": "%d-token stored document + %d fresh tokens" % (doc_tokens, suffix_tokens),
                     "pool_blocks": pool, "docs": n_docs, "iters": iters, "reserve_headroom": headroom,
                     "copy_bound": "bytes of the step's fetch and insert copies (read + write) / measured copy bandwidth"}
    st.close()
    return res


def lookup_fetch_cases(torch, st, cache, docs, rng, mb, suffix_tokens, peak, sh):
    """ptstore_lookup_fetch alone on 16-prompt batches that are not uniform: all prompts over ONE stored document (every
    block shared: read once, written 16 times) and one prompt that hits beside fifteen that miss.  Median of 10 calls,
    microseconds, next to the time the bytes DRAM must move (distinct blocks read + delivered blocks written) would take at
    the measured copy bandwidth."""
    import ctypes as C
    from paper_2607_22648_b200 import binding as G

    def dev(a):
        return torch.from_numpy(np.ascontiguousarray(a)).cuda()

    def fresh(n):
        return rng.integers(0, 128256, size=n, dtype=np.int32)

    cases = {
        "16_prompts_over_one_document": [np.concatenate([docs[0], fresh(suffix_tokens)]) for _ in range(16)],
        "1_prompt_hits_15_miss": [np.concatenate([docs[1], fresh(suffix_tokens)])] + [fresh(len(docs[1]) + suffix_tokens) for _ in range(15)],
        "16_prompts_over_16_documents": [np.concatenate([docs[i], fresh(suffix_tokens)]) for i in range(16)],
    }
    stream = torch.cuda.current_stream().cuda_stream
    out = {}
    for name, seqs in cases.items():
        toks, offs = W.ragged(seqs)
        t, o = dev(toks), dev(offs)
        bt = dev(rng.permutation(16 * mb).astype(np.int32).reshape(16, mb))
        matched = torch.empty(16, dtype=torch.int32, device="cuda")
        ids = torch.empty((16, mb), dtype=torch.int32, device="cuda")
        args = (st.h, t.data_ptr(), o.data_ptr(), 16, mb, 0, C.byref(cache.desc), bt.data_ptr(), matched.data_ptr(), ids.data_ptr(), stream)
        us = []
        s0 = None
        for k in range(13):
            if k == 3:
                s0 = st.stats()
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record(); assert G.lib.ptstore_lookup_fetch(*args) == 0; b.record(); torch.cuda.synchronize()
            if k >= 3:
                us.append(a.elapsed_time(b) * 1e3)
        s1 = st.stats()
        delivered = (s1.blocks_fetched[0] - s0.blocks_fetched[0]) / 10
        distinct = (s1.blocks_fetched_distinct - s0.blocks_fetched_distinct) / 10
        need = (delivered + distinct) * sh.block_bytes
        out[name] = {"call_us": round(float(np.median(us)), 1), "blocks_delivered": delivered, "blocks_read": distinct,
                     "dram_bound_us": round(need / (peak * 1e9) * 1e6, 1), "call_over_bound": round(float(np.median(us)) / (need / (peak * 1e9) * 1e6), 3)}
    assert st.status() == 0
    return out


def ceilings_record(torch, writes_x100=274, gib=4):
    """What the bulk copy engine itself reaches on this GPU, by traffic pattern (ptstore_copy_probe over plain buffers larger
    than L2, the ring the store uses for 32 KiB chunks, best of 4 launches each): loads only, stores only, a 1:1 copy, and
    the read-once-write-many mix of the benchmark's fetch."""
    from paper_2607_22648_b200 import binding as G
    n = gib << 30
    w = (writes_x100 + 99) // 100
    src = torch.empty(n, dtype=torch.uint8, device="cuda").fill_(3)
    dst = torch.empty(n * w, dtype=torch.uint8, device="cuda").fill_(5)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = {}
    for name, mode, moved in (("read_only", G.PROBE_READ, n), ("write_only", G.PROBE_WRITE, n), ("copy_1to1", G.PROBE_COPY, 2 * n),
                              ("mix_1to%.2f" % (writes_x100 / 100), G.PROBE_MIX, n + n * writes_x100 / 100)):
        best = 1e9
        for r in range(5):
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record()
            G.copy_probe(src, dst, n, mode, writes_x100, status=status)
            b.record(); torch.cuda.synchronize()
            if r:
                best = min(best, a.elapsed_time(b))
        out[name] = round(moved / (best * 1e-3) / 1e9, 1)
    # the same 1:1 copy with four stages: more loads in flight help the loads and cost the copy
    for name, mode, moved in (("read_only_4_stages", G.PROBE_READ, n), ("copy_1to1_4_stages", G.PROBE_COPY, 2 * n)):
        best = 1e9
        for r in range(4):
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record()
            G.copy_probe(src, dst, n, mode, writes_x100, stages=4, status=status)
            b.record(); torch.cuda.synchronize()
            if r:
                best = min(best, a.elapsed_time(b))
        out[name] = round(moved / (best * 1e-3) / 1e9, 1)
    assert int(status.item()) == 0
    out["unit"] = "GB/s (bytes read + bytes written)"
    out["how"] = "ptstore_copy_probe, 3 stages x 32 KiB, 1 CTA per SM, %d GiB read per launch, paged-cache-like destinations" % gib
    return out


def run_latency(args):
    import torch
    torch.cuda.set_device(0)
    from __graft_entry__ import build
    build()
    sampler = ClockSampler(0)
    sampler.start()
    kw = {}
    if args.batch:                        # a small case (for a profiler): one batch size, fewer stored documents
        kw["batches"] = (args.batch,)
    if args.docs:
        kw["n_docs"] = args.docs
    rec = latency_record(args, torch, iters=max(args.steps, 10), **kw)
    clocks = sampler.stop()
    b1 = rec["batch%d" % (args.batch or 1)]
    peak, kind = measured_peak()
    out = {"metric": "prefix-hit KV fetch GB/s", "value": b1["gbps"], "unit": "GB/s", "n_gpus": 1, "steps": rec["config"]["iters"], "warmup": 8,
           "ms_per_step": round(b1["step_us"] / 1e3, 4), "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
           "data": "synthetic", "config": dict(rec["config"], workload="latency_llama3_8b_4k_prompt_full_hit_batch" + "_".join(str(b) for b in kw.get("batches", (1, 4, 16))),
                          l2="512 MiB of KV per prompt: larger than L2"),
           "latency": rec, "gpu_launches": int(b1["launches_per_step"] * rec["config"]["iters"]), "clocks": clocks,
           "roofline": {"bound": "hbm", "kernel": "whole batch-%d step" % (args.batch or 1), "achieved": b1["gbps"], "peak": peak, "unit": "GB/s",
                        "frac": round(b1["gbps"] / peak, 4), "traffic": None, "peak_kind": kind + " (plain copy, read+write)"}}
    print(json.dumps(out), flush=True)


# ---------------------------------------------------------------------------------------------------------
def lookup_record(args, torch, K=200, W_=5, variants=None):
    """configs[2]: lookup-only stress.  One call = ptstore_lookup over 16,384 requests x 64 blocks against a 10^6-node trie at
    load factor 0.7; K calls run back to back between two events (table and tokens warm in L2), then 10 more with L2
    flushed before each."""
    from paper_2607_22648_b200 import binding as G
    ws = W.lookup_stress()
    wa = W.lookup_stress(all_hit=True)
    sh = W.KVShape(1, 1, 8, 16)
    st = G.PTStore(sh.layers, sh.heads, sh.dim, sh.block_tokens, ws.n_nodes, max_requests=16384, max_batch_blocks=16384 * 64,
                   table_slots=ws.table_slots, flags=G.lookup_lanes(args.lanes))

    def dev(a):
        return torch.from_numpy(np.ascontiguousarray(a)).cuda()

    for i in range(0, len(ws.store_seqs), 8192):
        t, o = W.ragged(ws.store_seqs[i:i + 8192])
        st.insert(dev(t), dev(o), 16)
    assert st.status() == 0
    res = {}
    matched = torch.empty(16384, dtype=torch.int32, device="cuda")
    ids = torch.empty((16384, 64), dtype=torch.int32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    sampler = ClockSampler(0)
    clocks = None
    todo = (("geometric_hit_depth", ws, 0), ("geometric_no_touch", ws, G.NO_TOUCH), ("geometric_pin", ws, G.PIN), ("all_hit", wa, G.NO_TOUCH))
    for name, wl, flags in todo:
        if variants and name not in variants:
            continue
        t, o = W.ragged(wl.queries)
        mb = W.max_blocks_of(wl.queries, 16)
        dt, do = dev(t), dev(o)
        m2, i2 = (matched, ids) if mb == 64 else (matched, torch.empty((16384, mb), dtype=torch.int32, device="cuda"))
        # the timed loop calls the C entry point directly with pre-marshalled arguments: a lookup takes tens of
        # microseconds, so per-call Python work (tensor attribute lookups, stream object creation) would be measured otherwise
        stream = torch.cuda.current_stream().cuda_stream
        cargs = (st.h, dt.data_ptr(), do.data_ptr(), 16384, mb, flags, m2.data_ptr(), i2.data_ptr(), stream)
        call = G.lib.ptstore_lookup
        for _ in range(W_):
            call(*cargs)
        s0 = st.stats()
        l0 = st.launch_count()
        if name == "geometric_hit_depth":
            sampler.start()
        # (a) back to back, table and tokens warm in L2
        torch.cuda.synchronize()
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        a.record()
        t0 = time.perf_counter()
        for _ in range(K):
            call(*cargs)
        host_us = (time.perf_counter() - t0) / K * 1e6
        b.record(); torch.cuda.synchronize()
        warm_ms = a.elapsed_time(b) / K
        if name == "geometric_hit_depth":
            clocks = sampler.stop()
        s1 = st.stats()
        launches = st.launch_count() - l0
        # (b) L2 flushed before every call
        cold = []
        for _ in range(min(K, 10)):
            flush.fill_(1)
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record(); call(*cargs); b.record(); torch.cuda.synchronize()
            cold.append(a.elapsed_time(b))
        if flags & G.PIN:
            for _ in range(W_ + K + len(cold)):
                st.release(i2, m2)
        q = (s1.query_blocks - s0.query_blocks) / K
        pr = (s1.probes_issued - s0.probes_issued) / K
        res[name] = {"ms_warm": round(warm_ms, 5), "ms_l2_flushed": round(float(np.median(cold)), 5),
                     "query_blocks_per_s": round(q / (warm_ms * 1e-3)), "issued_probes_per_s": round(pr / (warm_ms * 1e-3)),
                     "matched_blocks_per_s": round((s1.blocks_matched - s0.blocks_matched) / K / (warm_ms * 1e-3)),
                     "issued_probes": pr, "query_blocks": q, "slots_per_probe": round((s1.slots_visited - s0.slots_visited) / K / max(pr, 1), 3),
                     "launches": launches, "calls": K, "host_us_per_call": round(host_us, 2)}
    assert st.status() == 0
    st.close()
    main = res.get("geometric_hit_depth") or next(iter(res.values()))
    summary = {"workload": "lookup_stress_1M_nodes_load0.7_16384x64_geometric0.9", "calls": K,
               "query_blocks_per_s": main["query_blocks_per_s"], "issued_probes_per_s": main["issued_probes_per_s"],
               "slots_per_probe": main["slots_per_probe"], "ms_warm": main["ms_warm"], "ms_l2_flushed": main["ms_l2_flushed"],
               "l2_sectors_per_probe": L2_SECTORS_PER_PROBE, "l2_sectors_per_probe_kind": "modelled: from the ncu capture of this kernel in profiles/",
               "all_hit_issued_probes_per_s": res["all_hit"]["issued_probes_per_s"] if "all_hit" in res else None,
               "all_hit_ms_warm": res["all_hit"]["ms_warm"] if "all_hit" in res else None}
    return {"variants": res, "summary": summary, "clocks": clocks}


def run_lookup(args):
    import torch
    torch.cuda.set_device(0)
    from __graft_entry__ import build
    build()
    K, W_ = args.steps, args.warmup
    rec = lookup_record(args, torch, K, W_)
    res = rec["variants"]
    main = res["geometric_hit_depth"]
    peak, kind = measured_peak()
    # algorithmic bytes of one call: tokens of the hashed blocks (64 B each), one 32-byte sector per probe, 4 B id per query block
    alg = main["issued_probes"] * (64 + 32) + main["query_blocks"] * 4 + 16384 * 12
    out = {"metric": "lookup probes/s", "value": main["query_blocks_per_s"], "unit": "query blocks/s", "n_gpus": 1, "steps": K, "warmup": W_,
           "ms_per_step": main["ms_warm"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64",
           "data": "synthetic",
           "config": {"workload": "lookup_stress_1M_nodes_load0.7_16384x64_geometric0.9", "lanes_per_request": args.lanes or "auto",
                      "l2": "table (22.9 MB) is L2 resident by design; ms_l2_flushed gives the cold figure"},
           "variants": res, "lookup": rec["summary"], "gpu_launches": main["launches"], "clocks": rec["clocks"],
           "roofline": {"bound": "hbm", "kernel": "lookup_kernel", "achieved": round(alg / (main["ms_warm"] * 1e-3) / 1e9, 1), "peak": peak,
                        "unit": "GB/s", "frac": round(alg / (main["ms_warm"] * 1e-3) / 1e9 / peak, 4), "traffic": None,
                        "note": "latency/issue bound, not bandwidth bound: the figure is context only"}}
    print(json.dumps(out), flush=True)


# ---------------------------------------------------------------------------------------------------------
def cpu_oracle_sample(args, steps=8, batch=8, pool_blocks=2800):
    """The CPU oracle, as it stands, on a bounded sample of the same stream: the same step on the same KV
    shape with `batch` prompts per step and a pool of `pool_blocks` blocks, real bytes moved with memcpy."""
    from oracle import Oracle, PIN
    sh = W.LLAMA3_8B
    stream = W.llama8b_stream(n_docs=args.docs or 500)
    o = Oracle(sh.layers, sh.heads, sh.dim, sh.elem_bytes, sh.block_tokens, 0, pool_blocks, 0, byte_mode=True)
    mb = stream.max_blocks
    B = sh.block_tokens
    rng = np.random.default_rng(5)
    batches = [stream.batch(batch)[0] for _ in range(steps + 1)]
    need_max = max(sum(len(s) // B for s in b) for b in batches)
    cache = o.new_cache(need_max + 1, fill=3)
    moved, moved_delivered, t_total = 0, 0, 0.0
    for k, seqs in enumerate(batches):
        toks, offs = W.ragged(seqs)
        bt = W.shuffled_block_tables(rng, seqs, B, mb, need_max + 1)
        t0 = time.perf_counter()
        m, ids = o.lookup(toks, offs, mb, PIN)
        o.fetch(ids, m, cache, bt)
        need = sum(len(s) // B for s in seqs) - int(m.sum())
        short = need - o.free_count(0)
        if short > 0:
            o.evict(0, short, literal=False)
        ins, newb = o.insert(toks, offs, mb, cache, bt)
        o.release(ids, m)
        dt = time.perf_counter() - t0
        if k == 0:
            continue                                     # first step only fills the pool
        t_total += dt
        hit = ids[np.arange(mb)[None, :] < m[:, None]]
        # the same byte count as the GPU arm's `value`: each distinct source block read once, each delivered block written, each
        # stored block read and written (the oracle itself copies every delivered block separately)
        moved += (len(np.unique(hit)) + int(m.sum()) + 2 * int(newb.sum())) * sh.block_bytes
        moved_delivered += (int(m.sum()) + int(newb.sum())) * 2 * sh.block_bytes
    o.close()
    return {"value": round(moved / t_total / 1e9, 2), "value_delivered_bytes": round(moved_delivered / t_total / 1e9, 2), "unit": "GB/s", "cores": 1, "kind": "oracle",
            "sample": "%d steps of %d prompts of the same document stream, pool %d blocks (%.1f GB), same step sequence; eviction by the "
                      "sorted closed form" % (steps, batch, pool_blocks, pool_blocks * sh.block_bytes / 1e9),
            "ms_per_step": round(t_total / steps * 1e3, 1), "host_cores_available": os.cpu_count()}


def cpu_oracle_threads_sample(args, steps=8, batch=16, pool_blocks=2800):
    """The oracle's read-only half of the step (lookup without stamps or pins, then the fetch) with the requests split
    over every hardware thread; insert and eviction stay sequential and are not part of this figure."""
    from oracle import Oracle
    sh = W.LLAMA3_8B
    stream = W.llama8b_stream(n_docs=args.docs or 500)
    o = Oracle(sh.layers, sh.heads, sh.dim, sh.elem_bytes, sh.block_tokens, 0, pool_blocks, 0, byte_mode=True)
    mb, B = stream.max_blocks, sh.block_tokens
    rng = np.random.default_rng(6)
    threads = os.cpu_count() or 1
    batches = [stream.batch(batch)[0] for _ in range(steps + 1)]
    need_max = max(sum(len(s) // B for s in b) for b in batches)
    cache = o.new_cache(need_max + 1, fill=3)
    moved, t_total = 0, 0.0
    for k, seqs in enumerate(batches):
        toks, offs = W.ragged(seqs)
        bt = W.shuffled_block_tables(rng, seqs, B, mb, need_max + 1)
        t0 = time.perf_counter()
        m, ids = o.lookup_fetch_threads(toks, offs, mb, cache, bt, threads)
        dt = time.perf_counter() - t0
        short = sum(len(s) // B for s in seqs) - int(m.sum()) - o.free_count(0)
        if short > 0:
            o.evict(0, short, literal=False)
        o.insert(toks, offs, mb, cache, bt)                # untimed: keeps the pool turning over as in the real step
        if k == 0:
            continue
        t_total += dt
        hit = ids[np.arange(mb)[None, :] < m[:, None]]
        moved += (len(np.unique(hit)) + int(m.sum())) * sh.block_bytes
    o.close()
    return {"value": round(moved / max(t_total, 1e-9) / 1e9, 2), "unit": "GB/s", "cores": threads, "kind": "oracle",
            "sample": "lookup + fetch only (the read-only phases), %d steps of %d prompts of the same document stream split over %d "
                      "threads, pool %d blocks" % (steps, batch, threads, pool_blocks),
            "ms_per_step": round(t_total / steps * 1e3, 1)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import build_oracle
    build_oracle()
    W_, K = args.warmup, args.steps
    res = cpu_oracle_sample(args, steps=max(K, 1))
    out = {"impl": "reference", "metric": "prefix-hit KV fetch GB/s", "value": res["value"], "unit": "GB/s",
           "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": K, "warmup": W_, "ms_per_step": res["ms_per_step"],
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
           "config": {"workload": "llama3_8b_kv_pool20k_zipf1.1_batch64", "note": "CPU oracle on a bounded sample of the workload"},
           "cpu_baseline": res, "e2e": {"value": res["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--engine", default="bulk", choices=["vector", "bulk"])
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--ctas-per-sm", type=int, default=0)
    ap.add_argument("--fill", type=int, default=6, help="untimed steps that fill the pool before warm-up")
    ap.add_argument("--workload", default="llama8b", choices=["llama8b", "llama70b", "churn", "lookup", "multiturn", "latency"])
    ap.add_argument("--block-tokens", type=int, default=0, help="llama8b workload: tokens per block (default 16)")
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--docs", type=int, default=0)
    ap.add_argument("--pool-blocks", type=int, default=0)
    ap.add_argument("--host-gb", type=float, default=0.0)
    ap.add_argument("--policy", default="lru", choices=["lru", "gdsf"], help="eviction order")
    ap.add_argument("--async-demote", action="store_true", help="churn workload: reserve before fetch, demotion copy on the side stream")
    ap.add_argument("--promote", type=int, default=0, help="churn workload: host-tier blocks promoted into HBM per step (budget)")
    ap.add_argument("--lanes", type=int, default=0, help="lookup workload: lanes per request (0 = library default)")
    ap.add_argument("--lookup-calls", type=int, default=200, help="back-to-back lookup calls of the lookup record")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-latency", action="store_true", help="skip the small-batch latency record")
    ap.add_argument("--no-lookup", action="store_true", help="skip the lookup stress record")
    ap.add_argument("--no-ceilings", action="store_true", help="skip the copy-engine ceiling probes")
    ap.add_argument("--stub-cpu", action="store_true", help="replica launch and aggregation on CPU with a stub step (tests)")
    ap.add_argument("--traffic", type=float, default=None, help="ncu DRAM bytes per fetch launch, if known (see profiles/)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        relaunch_as_replicas(args)                        # does not return
    if args.stub_cpu:
        run_stub_replicas(args)
    elif args.workload == "lookup":
        run_lookup(args)
    elif args.workload == "latency":
        run_latency(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
