#!/usr/bin/env python
"""Benchmark of the AQ-SGD boundary codec on B200.

Headline workload (default): the GPT2-1.5B-shaped boundary -- hidden 1600, sequence 1024,
micro-batch 1, fp16, 4-bit deltas, group 64, 4096 sample ids per side (13.4 GB of m on
the sender and again on the receiver), a fresh seeded id order per epoch.  One STEP is one
macro-batch of 32 micro-batches (the paper's GPT2 setting) crossing the boundary:
aq_encode on the sender handle, then aq_decode on the receiver handle.  Epoch 0 (first
visits, uncompressed) is run and timed apart; the timed steps are steady-state delta visits
of later epochs, whose activations are generated into HBM before the clock starts.

The timed region of `--steps` K steps is repeated (at least 30 windows, and until half a
second of GPU time is covered); `ms_per_step` is the median window, with minimum, maximum
and the number of windows beside it.

One JSON line on stdout (rank 0).  `value` = algorithmic GB/s of encode+decode over the
timed steps of all ranks; `roofline` = the encode kernel against the measured HBM copy
peak; `e2e` = the same step through aq_encode_host / aq_decode_host with pinned host
buffers; `cpu_baseline` = the CPU oracle on a bounded sample of the same workload, on one
core and on all host cores; `configs` (one GPU only) = the same measurement for the
DeBERTa-1.5B-shaped boundary, one boundary of the pipeline sweep and the backward path, each
also with calls of the workload's own micro-batch size.

`--impl reference` times the CPU oracle instead (rank 0 only).
"""
import argparse
import hashlib
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# name -> (recipe in fixtures.synth, sequences per macro-batch, label); the paper's GPT2 runs use macro-batch 32 of
# micro-batch 1, its DeBERTa/QNLI runs macro-batch 64 of micro-batch 8
WORKLOADS = {"gpt2": ("GPT2_XL", 32, "GPT2-1.5B-shaped boundary (configs[1])"),
             "deberta": ("DEBERTA_XXL", 64, "DeBERTa-1.5B-shaped boundary (configs[2])"),
             # one of the 8 boundaries of the pipeline sweep (they are independent and alike): per macro-batch of 16
             # micro-batches, forward 3-bit deltas and backward 6-bit gradients, each over a device-to-device wire
             "sweep": ("SWEEP_FWD", 16, "one boundary of the pipeline sweep (configs[4]): fwd 3-bit delta + bwd 6-bit direct + wire copies")}
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic of one delta-visit launch from an ncu capture (dram__bytes_read.sum + dram__bytes_write.sum),
# per element, by workload; reported as roofline.traffic only while the kernel sources still hash to the
# value recorded with the capture (`python bench.py --kernel-hash` prints the current one).
NCU_TRAFFIC = {
    "gpt2": {"kernel_hash": "cd123e3688cfb3ef", "encode_bytes_per_element": (209772800 + 77900544) / 52428800,
             "capture": "ncu --set full, encode_kernel<__half,4,8,0>, one launch of 32 sequences on the 128-id case"},
}


def kernel_source_hash():
    """SHA-256 (first 16 hex digits) over the kernel sources that the traffic figures were taken from."""
    h = hashlib.sha256()
    for name in ("aq_internal.h", "aq_device.cuh", "aq_kernels.cu"):
        with open(os.path.join(ROOT, "paper_2206_01299_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default="gpt2", choices=sorted(WORKLOADS), help="the headline workload")
    ap.add_argument("--configs", default=None, choices=["all", "headline"],
                    help="all (default on one GPU): also measure the other workloads, reported under `configs`")
    ap.add_argument("--topology", default="replicas", choices=["replicas", "pipeline"],
                    help="replicas (default): every rank runs both sides of its own boundary.  pipeline (an even number of "
                         "ranks): ranks 2p and 2p+1 are the sending and the receiving stage of boundary p, the message "
                         "travels between them through torch.distributed (paper_2206_01299_b200.link)")
    ap.add_argument("--backend", default="nccl", choices=["nccl", "gloo"],
                    help="process-group backend for N > 1.  gloo lets several ranks share one GPU (rank -> device "
                         "rank %% device count): a functional check of the multi-rank paths where only one GPU is at hand")
    ap.add_argument("--n-samples", type=int, default=None, help="shrink the id space (profiling runs)")
    ap.add_argument("--per-launch", type=int, default=0, help="sequences handed to one aq_encode call (0 = the whole macro-batch)")
    ap.add_argument("--graph", action="store_true", help="replay each step as a captured CUDA graph")
    ap.add_argument("--rounding", default="interval", choices=["interval", "stochastic"],
                    help="quantizer of the sender: interval number (default) or unbiased stochastic rounding")
    ap.add_argument("--m-bits", type=int, default=0, choices=[0, 2, 4, 8, 32],
                    help="keep the previous messages in this many bits per element (0 = the activation type, 32 = binary32)")
    ap.add_argument("--hosted", action="store_true", help="keep m in page-locked host memory (aq_create_hosted)")
    ap.add_argument("--prefetch", action="store_true",
                    help="with --hosted: fetch every call's previous messages ahead of it (aq_prefetch); the calls "
                         "then run on staged rows in HBM and write them back behind the caller")
    ap.add_argument("--stage-compute-ms", type=float, default=0.0,
                    help="with --hosted: a stand-in for the stage's own work, a kernel that holds the handles' stream "
                         "for about this many ms after every step (what of the transfers stays on the critical path)")
    ap.add_argument("--min-timed-ms", type=float, default=500.0, help="repeat the timed region until it covers this much GPU time")
    ap.add_argument("--max-repeats", type=int, default=400)
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-aux", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=32)
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--kernel-hash", action="store_true", help="print the hash of the kernel sources and exit")
    return ap.parse_args()


def bytes_per_element(bits, group, m_bits=0):
    """Algorithmic HBM bytes per element of a steady-state encode (= of a decode):
    read a (2) + read m (2) + write m (2) + codes (b/8) + scale (4/G); with m kept in z bits:
    a (2) + m read and written (2 * (z/8 + 4/G)) + codes (b/8) + scale (4/G)."""
    if m_bits == 32:                                  # binary32 store: no steps
        return 2.0 + 8.0 + bits / 8.0 + 4.0 / group
    if m_bits:
        return 2.0 + 2.0 * (m_bits / 8.0 + 4.0 / group) + bits / 8.0 + 4.0 / group
    return 6.0 + bits / 8.0 + 4.0 / group


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.dev = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.dev, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _names(self, mask):
        nv, out = self.nv, []
        table = [("hw_slowdown", "nvmlClocksThrottleReasonHwSlowdown"),
                 ("hw_thermal_slowdown", "nvmlClocksThrottleReasonHwThermalSlowdown"),
                 ("sw_thermal_slowdown", "nvmlClocksThrottleReasonSwThermalSlowdown"),
                 ("sw_power_cap", "nvmlClocksThrottleReasonSwPowerCap"),
                 ("hw_power_brake", "nvmlClocksThrottleReasonHwPowerBrakeSlowdown")]
        for name, attr in table:
            bit = getattr(nv, attr, 0)
            if bit and (mask & bit):
                out.append(name)
        return out

    def _sample(self):
        nv = self.nv
        try:
            self.samples.append(nv.nvmlDeviceGetClockInfo(self.dev, nv.NVML_CLOCK_SM))
            self.reasons.update(self._names(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.dev)))
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self._sample()
            time.sleep(0.002)

    def __enter__(self):
        if self.nv:
            # the timed loop keeps the interpreter busy; a short switch interval lets this thread in
            self._switch = sys.getswitchinterval()
            sys.setswitchinterval(0.0005)
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread:
            self._thread.join()
            sys.setswitchinterval(self._switch)
            self._sample()                                    # a very short timed region still gets a reading at its end

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def bits16(t):
    import numpy as np
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


# ------------------------------------------------------------------------------------ CPU oracle timing

def time_oracle(cfg, budget_s, device, max_samples=256):
    """Steady-state encode + decode of whole samples by the CPU oracle, as it stands, until
    about budget_s seconds of work are done.  Returns (GB/s, samples/s, n_samples, seconds)."""
    import numpy as np
    import oracle
    from fixtures import synth
    od = oracle.FP16 if cfg.dtype == "fp16" else oracle.BF16
    small = synth.shrink(cfg, max_samples)
    snd = oracle.Side(max_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group, od)
    rcv = oracle.Side(max_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group, od)
    done, spent = 0, 0.0
    while done < max_samples and (spent < budget_s or done < 2):
        ids = np.array([done], np.int32)
        a0 = bits16(synth.activation(small, [done], 0, device=device))
        a1 = bits16(synth.activation(small, [done], 1, device=device))
        p, s, _ = snd.encode(a0, ids)                 # first visit, untimed
        rcv.decode(p, s, ids, raw=a0)
        t0 = time.perf_counter()
        p, s, _ = snd.encode(a1, ids)
        rcv.decode(p, s, ids)
        spent += time.perf_counter() - t0
        done += 1
    gb = 2 * done * cfg.elems * bytes_per_element(cfg.bits, cfg.group) / 1e9
    return gb / spent, done / spent, done, spent


def _oracle_worker(job):
    """One process of the all-cores leg: the unchanged single-threaded oracle on this worker's own
    samples (first visits untimed), then, once every worker is ready, delta visits that alternate
    between two epochs of each sample until the budget is spent.  Returns (visits, seconds)."""
    path, which, shape, bits, group, dtype, budget_s, ready_at = job
    import numpy as np
    import oracle
    n_ids, seq, hidden = len(which), shape[0], shape[1]
    acts = np.load(path, mmap_mode="r")                          # [n_pool, 2, seq, hidden] uint16
    mine = [np.ascontiguousarray(acts[w]) for w in which]
    snd = oracle.Side(n_ids, seq, hidden, bits, group, dtype)
    rcv = oracle.Side(n_ids, seq, hidden, bits, group, dtype)
    for j in range(n_ids):
        ids = np.array([j], np.int32)
        p, s, _ = snd.encode(mine[j][0:1], ids)
        rcv.decode(p, s, ids, raw=mine[j][0:1])
    while time.time() < ready_at:                                # every worker starts its timed visits together
        time.sleep(0.005)
    visits, t0 = 0, time.perf_counter()
    while time.perf_counter() - t0 < budget_s:
        j, e = visits % n_ids, 1 - (visits // n_ids) % 2
        ids = np.array([j], np.int32)
        p, s, _ = snd.encode(mine[j][e:e + 1], ids)
        rcv.decode(p, s, ids)
        visits += 1
    return visits, time.perf_counter() - t0


def time_oracle_all_cores(cfg, budget_s, device):
    """The same oracle, one worker process per host core, no threading inside it: every worker
    visits its own samples.  Returns a dict for cpu_baseline.all_cores."""
    import multiprocessing as mp
    import tempfile
    import numpy as np
    import oracle
    from fixtures import synth
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    per_worker = 2
    pool_ids = min(per_worker * cores, 64)                       # bounded input set: workers beyond 32 share samples
    small = synth.shrink(cfg, pool_ids)
    acts = np.empty((pool_ids, 2, cfg.seq, cfg.hidden), np.uint16)
    for i in range(pool_ids):
        for e in (0, 1):
            acts[i, e] = bits16(synth.activation(small, [i], e, device=device))[0]
    od = oracle.FP16 if cfg.dtype == "fp16" else oracle.BF16
    with tempfile.TemporaryDirectory() as tmp:
        path = os.path.join(tmp, "acts.npy")
        np.save(path, acts)
        ready_at = time.time() + 6.0 + 0.02 * cores               # start-up of the workers (imports, first visits)
        jobs = [(path, [(per_worker * w + j) % pool_ids for j in range(per_worker)], (cfg.seq, cfg.hidden), cfg.bits,
                 cfg.group, od, budget_s, ready_at) for w in range(cores)]
        ctx = mp.get_context("spawn")
        with ctx.Pool(cores) as pool:
            got = pool.map(_oracle_worker, jobs, chunksize=1)
    visits = sum(v for v, _ in got)
    secs = max(s for _, s in got)
    gb = 2 * visits * cfg.elems * bytes_per_element(cfg.bits, cfg.group) / 1e9
    return {"value": gb / secs, "unit": "GB/s", "cores": cores, "samples_per_s": visits / secs,
            "sample": f"{cores} worker processes (one per host core, nproc = {cores}), each the single-threaded oracle on "
                      f"{per_worker} whole sequences of its own ({pool_ids} distinct sequences in all), steady-state "
                      f"encode+decode visits for {budget_s:.0f} s: {visits} visits"}


def run_reference(args, cfg):
    """The oracle as the reference arm: each step = steady-state encode + decode of `rows`
    token rows of one sample (a bounded sample of the macro-batch step), on one host core."""
    import numpy as np
    import torch
    import oracle
    from fixtures import synth
    device = "cuda" if torch.cuda.is_available() else "cpu"
    # calibrate on one full sample, then size the per-step sample so the run stays near two minutes
    _, sps, _, _ = time_oracle(cfg, 0.0, device, max_samples=2)
    per_sample_s = 1.0 / sps
    total = args.steps + args.warmup
    rows = int(max(8, min(cfg.seq, cfg.seq * (120.0 / total) / per_sample_s)))
    sub = synth.shrink(cfg, 8, seq=rows)
    od = oracle.FP16 if cfg.dtype == "fp16" else oracle.BF16
    snd = oracle.Side(8, rows, cfg.hidden, cfg.bits, cfg.group, od)
    rcv = oracle.Side(8, rows, cfg.hidden, cfg.bits, cfg.group, od)
    acts = {}
    for sid in range(8):
        for ep in range(0, 5):
            acts[(sid, ep)] = bits16(synth.activation(sub, [sid], ep, device=device))
        ids = np.array([sid], np.int32)
        p, s, _ = snd.encode(acts[(sid, 0)], ids)
        rcv.decode(p, s, ids, raw=acts[(sid, 0)])
    elapsed = 0.0
    for step in range(total):
        sid, ep = step % 8, 1 + (step // 8) % 4
        ids = np.array([sid], np.int32)
        t0 = time.perf_counter()
        p, s, _ = snd.encode(acts[(sid, ep)], ids)
        rcv.decode(p, s, ids)
        dt = time.perf_counter() - t0
        if step >= args.warmup:
            elapsed += dt
    elems = rows * cfg.hidden
    gbs = 2 * args.steps * elems * bytes_per_element(cfg.bits, cfg.group) / 1e9 / elapsed
    sample = f"{rows} of {cfg.seq} token rows of one sequence per step ({elems} elements), steady-state encode+decode"
    line = {
        "impl": "reference", "metric": "activation encode+decode GB/s", "value": gbs, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": elapsed / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOADS[args.workload][2] + ", CPU oracle on a bounded sample",
                   "hidden": cfg.hidden, "seq": cfg.seq, "bits": cfg.bits, "group": cfg.group,
                   "act_dtype": cfg.dtype},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------ GPU arm

class Env:
    """What every measurement needs: the process's rank, the process group (or None), the stream."""

    def __init__(self, rank, local_rank, world, dist, stream):
        self.rank, self.local_rank, self.world, self.dist, self.stream = rank, local_rank, world, dist, stream


def measure_boundary(args, env, name, steps, warmup, headline):
    """One forward boundary at full size (or --n-samples): first-visit epoch, `repeats` timed windows of
    `steps` steady-state steps, per-kernel durations, calls of the workload's own micro-batch size, and for
    the headline workload the isolated-call, end-to-end and remaining-kernel figures.  Returns a dict; the
    handles and every buffer are gone when it returns."""
    import numpy as np
    import torch
    from dataclasses import replace
    import paper_2206_01299_b200 as aq
    from fixtures import replicas, synth

    rank, local_rank, world, dist, stream = env.rank, env.local_rank, env.world, env.dist, env.stream
    recipe, macro, label = WORKLOADS[name]
    cfg = getattr(synth, recipe)
    if args.n_samples:
        cfg = synth.shrink(cfg, args.n_samples)
    # data-parallel replicas: every rank owns its own id shard of a world-times larger id space (weak
    # scaling); sample rows never cross ranks, so the data path has no collective
    cfg = replicas.shard_for_rank(cfg, rank, world)
    m_bits = args.m_bits if headline else 0
    hosted, prefetching = (args.hosted, args.prefetch) if headline else (False, False)
    stochastic = headline and args.rounding == "stochastic"
    use_graph = headline and args.graph

    nb = (args.per_launch if headline else 0) or macro
    assert cfg.n_samples % macro == 0 and macro % nb == 0
    steps_per_epoch = cfg.n_samples // macro
    launches_per_step = macro // nb
    # resident steady-state epochs: at most 4 (2 for the 26 GB boundaries), fewer when the id space is small
    max_arenas = 4 if cfg.n_samples * cfg.elems * 2 < 20e9 else 2
    n_arenas = max(1, min(max_arenas, (steps + warmup + steps_per_epoch - 1) // steps_per_epoch))
    bpe = bytes_per_element(cfg.bits, cfg.group, m_bits)
    step_bytes = 2 * macro * cfg.elems * bpe          # encode + decode

    def create():
        h = (aq.aq_create_hosted_lowbit(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group, m_bits) if m_bits in (2, 4, 8) and hosted
             else aq.aq_create_fp32(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group) if m_bits == 32
             else aq.aq_create_lowbit(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group, m_bits) if m_bits
             else aq.aq_create_hosted(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group) if hosted
             else aq.aq_create(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group))
        aq.aq_configure(h, aq.AQ_DTYPE, aq.AQ_FP16 if cfg.dtype == "fp16" else aq.AQ_BF16)
        aq.aq_configure(h, aq.AQ_BATCH, nb)
        aq.aq_configure(h, aq.AQ_STREAM, stream.cuda_stream)
        if stochastic:
            aq.aq_configure(h, aq.AQ_ROUNDING, aq.AQ_ROUND_STOCHASTIC)
            aq.aq_configure(h, aq.AQ_SEED, 20220601)
        return h

    snd, rcv = create(), create()
    handles = [snd, rcv]

    # fp32 running sum A_e of every sample in id order (the recipe's state), advanced one epoch at a time;
    # id spaces too large for that (4 B per element beside the two m arrays) recompute A_e per chunk instead
    keep_running = cfg.n_samples * cfg.elems * 4 < 40e9
    running = torch.empty((cfg.n_samples, cfg.elems), dtype=torch.float32, device="cuda") if keep_running else None
    all_ids = torch.arange(cfg.n_samples)

    def gen_arena(epoch, order):
        """Activations of one epoch in visiting order: arena[p] = a(order[p]) at that epoch."""
        if not keep_running:
            arena = torch.empty((cfg.n_samples, cfg.seq, cfg.hidden), dtype=cfg.torch_dtype, device="cuda")
            for c in range(0, cfg.n_samples, 16):
                arena[c:c + 16] = synth.activation(cfg, order[c:c + 16], epoch, device="cuda")
            return arena
        for c in range(0, cfg.n_samples, 16):
            ids = all_ids[c:c + 16]
            if epoch == 0:
                running[c:c + 16] = synth.base_f32(cfg, ids, "cuda")
            else:
                running[c:c + 16] = synth.advance_f32(cfg, running[c:c + 16], ids, epoch)
        arena = torch.empty((cfg.n_samples, cfg.seq, cfg.hidden), dtype=cfg.torch_dtype, device="cuda")
        order_dev = order.cuda().long()
        for c in range(0, cfg.n_samples, 64):
            arena[c:c + 64] = running[order_dev[c:c + 64]].to(cfg.torch_dtype).reshape(-1, cfg.seq, cfg.hidden)
        return arena

    packed = torch.empty((macro, cfg.packed_bytes), dtype=torch.uint8, device="cuda")
    scales = torch.empty((macro, cfg.groups), dtype=torch.float32, device="cuda")
    # the receiver's output rotates over buffers that together exceed twice the L2, so that no launch finds the
    # lines it is about to overwrite still dirty in cache
    n_outs = max(2, math.ceil(2 * 126e6 / (macro * cfg.elems * 2)) + 1)
    outs = [torch.empty((macro, cfg.seq, cfg.hidden), dtype=cfg.torch_dtype, device="cuda") for _ in range(n_outs)]
    out = outs[0]

    sweep = name == "sweep"
    if sweep:
        # receiver's ends of the forward wire, both ends of the backward wire, rotating gradients (4 x 52 MB > L2)
        bw = synth.SWEEP_BWD
        bbits, n_grad = bw.bits[0], macro * cfg.elems
        rx_packed, rx_scales = torch.empty_like(packed), torch.empty_like(scales)
        grads = [synth.gradient(replace(bw, n_batch=macro), i, device="cuda") for i in range(4)]
        g_tx = (torch.empty(n_grad * bbits // 8, dtype=torch.uint8, device="cuda"), torch.empty(n_grad // bw.group, dtype=torch.float32, device="cuda"))
        g_rx = (torch.empty_like(g_tx[0]), torch.empty_like(g_tx[1]))
        g_outs = [torch.empty(n_grad, dtype=cfg.torch_dtype, device="cuda") for _ in range(n_outs)]
        grad_bytes = n_grad * (2 + bbits / 8 + 4 / bw.group)
        step_bytes += (2 * grad_bytes                                                  # quantize + dequantize
                       + 2 * (macro * (cfg.packed_bytes + cfg.groups * 4))             # forward wire: read + write
                       + 2 * (n_grad * bbits // 8 + n_grad // bw.group * 4))           # backward wire

    host_ids = {}                                      # device id list -> its host copy (aq_prefetch reads ids on the host)
    ahead = {"key": None}                              # the step whose rows were fetched at the end of the step before

    def prefetch(ids_dev, lo):
        key = ids_dev.data_ptr()
        if key not in host_ids:                        # once per id list: a device-to-host copy in the timed
            host_ids[key] = ids_dev.cpu()              # steps would queue behind the write-backs
        ih = host_ids[key][lo:lo + nb]
        aq.aq_prefetch(snd, ih)
        aq.aq_prefetch(rcv, ih)

    # stand-in for the stage's own work: a kernel that occupies the handles' stream for a fixed number of
    # clock cycles and draws next to no power, so that its duration does not depend on what runs beside it
    stage_cycles, stage_ms = 0, 0.0
    if headline and args.stage_compute_ms > 0:
        stage_cycles = int(args.stage_compute_ms * 1e-3 * 1.965e9)
        with torch.cuda.stream(stream):
            torch.cuda._sleep(stage_cycles)
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record(stream)
            for _ in range(4):
                torch.cuda._sleep(stage_cycles)
            c1.record(stream)
        torch.cuda.synchronize()
        stage_ms = c0.elapsed_time(c1) / 4

    def run_step(arena, ids_dev, s, raw=False, nxt=None):
        """One macro-batch: its micro-batches in launches of nb, each encoded then decoded (the pipeline
        sweep: encode, wire, decode, then the gradient of the macro-batch quantized, wired and dequantized).
        nxt = (ids_dev, s) of the step that follows: with --prefetch its rows are asked for as soon as this
        step's calls are issued, so that they travel while the stage computes."""
        for l in range(launches_per_step):
            lo = s * macro + l * nb
            a, i = arena[lo:lo + nb], ids_dev[lo:lo + nb]
            p, sc, o = packed[l * nb:(l + 1) * nb], scales[l * nb:(l + 1) * nb], outs[s % n_outs][l * nb:(l + 1) * nb]
            if prefetching and ahead["key"] != (ids_dev.data_ptr(), lo):
                prefetch(ids_dev, lo)
            aq.aq_encode(snd, a, i, p, sc)
            if raw:
                aq.aq_configure(rcv, aq.AQ_RAW, a)
            if sweep:
                rp, rs = rx_packed[l * nb:(l + 1) * nb], rx_scales[l * nb:(l + 1) * nb]
                aq.aq_wire_copy(snd, local_rank, rp, rs, None, p, sc, None)
                aq.aq_decode(rcv, rp, rs, i, o)
            else:
                aq.aq_decode(rcv, p, sc, i, o)
        ahead["key"] = None
        if prefetching and nxt is not None and launches_per_step == 1:
            prefetch(nxt[0], nxt[1] * macro)
            ahead["key"] = (nxt[0].data_ptr(), nxt[1] * macro)
        if stage_cycles:
            torch.cuda._sleep(stage_cycles)
        if sweep:
            aq.aq_quant_grad(rcv, grads[s % 4], n_grad, bbits, g_tx[0], g_tx[1])
            aq.aq_wire_copy_grad(rcv, local_rank, g_rx[0], g_rx[1], g_tx[0], g_tx[1], n_grad, bbits)    # the backward wire
            aq.aq_dequant_grad(snd, g_rx[0], g_rx[1], n_grad, bbits, g_outs[s % n_outs])

    ev = lambda: torch.cuda.Event(enable_timing=True)

    def kernel_pass(first_step, window):
        """Average duration of one encode launch and of one decode launch: `window` steps whose
        encode launches run back to back between one pair of events, then their decode launches
        between another (the wire buffers of the whole window are kept in between).  An event
        between every two launches would add about 2 us of idle stream time per event."""
        wp = torch.empty((window, macro, cfg.packed_bytes), dtype=torch.uint8, device="cuda")
        ws = torch.empty((window, macro, cfg.groups), dtype=torch.float32, device="cuda")
        e = [ev(), ev(), ev()]
        e[0].record(stream)
        for w in range(window):
            arena, ids_dev, s = step_source(first_step + w)
            for l in range(launches_per_step):
                lo = s * macro + l * nb
                aq.aq_encode(snd, arena[lo:lo + nb], ids_dev[lo:lo + nb], wp[w, l * nb:(l + 1) * nb], ws[w, l * nb:(l + 1) * nb])
        e[1].record(stream)
        for w in range(window):
            arena, ids_dev, s = step_source(first_step + w)
            for l in range(launches_per_step):
                lo = s * macro + l * nb
                aq.aq_decode(rcv, wp[w, l * nb:(l + 1) * nb], ws[w, l * nb:(l + 1) * nb], ids_dev[lo:lo + nb],
                             outs[w % n_outs][l * nb:(l + 1) * nb])
        e[2].record(stream)
        torch.cuda.synchronize()
        n = window * launches_per_step
        return e[0].elapsed_time(e[1]) / n, e[1].elapsed_time(e[2]) / n

    def grad_pass(window):
        """The same for the sweep's backward kernels: `window` quantize launches back to back, then
        `window` dequantize launches; gradients, wire buffers and outputs rotate over sets larger than L2."""
        n_tx = math.ceil(2 * 126e6 / (n_grad * bbits // 8)) + 1
        tx = [(torch.empty_like(g_tx[0]), torch.empty_like(g_tx[1])) for _ in range(n_tx)]
        for i in range(n_tx):
            aq.aq_quant_grad(rcv, grads[i % 4], n_grad, bbits, tx[i][0], tx[i][1])
        e = [ev(), ev(), ev()]
        e[0].record(stream)
        for w in range(window):
            aq.aq_quant_grad(rcv, grads[w % 4], n_grad, bbits, tx[w % n_tx][0], tx[w % n_tx][1])
        e[1].record(stream)
        for w in range(window):
            aq.aq_dequant_grad(snd, tx[w % n_tx][0], tx[w % n_tx][1], n_grad, bbits, g_outs[w % n_outs])
        e[2].record(stream)
        torch.cuda.synchronize()
        return e[0].elapsed_time(e[1]) / window, e[1].elapsed_time(e[2]) / window

    # one throw-away visit on a small boundary of the same type, bit width and group: the first launch of a
    # kernel loads its code (milliseconds), which must not count as first-visit time
    warm = [aq.aq_create_fp32(2, 8, cfg.hidden, cfg.bits, cfg.group) if m_bits == 32
            else aq.aq_create_lowbit(2, 8, cfg.hidden, cfg.bits, cfg.group, m_bits) if m_bits
            else aq.aq_create(2, 8, cfg.hidden, cfg.bits, cfg.group) for _ in range(2)]
    for h in warm:
        aq.aq_configure(h, aq.AQ_DTYPE, aq.AQ_FP16 if cfg.dtype == "fp16" else aq.AQ_BF16)
        aq.aq_configure(h, aq.AQ_STREAM, stream.cuda_stream)
        if stochastic:
            aq.aq_configure(h, aq.AQ_ROUNDING, aq.AQ_ROUND_STOCHASTIC)
    w_act = torch.zeros((1, 8, cfg.hidden), dtype=cfg.torch_dtype, device="cuda")
    w_ids = torch.zeros(1, dtype=torch.int32, device="cuda")
    aq.aq_configure(warm[1], aq.AQ_RAW, w_act)
    for _ in range(2):                                 # a first visit, then a delta visit
        aq.aq_encode(warm[0], w_act, w_ids, packed[:1], scales[:1])
        aq.aq_decode(warm[1], packed[:1], scales[:1], w_ids, out[:1])
    torch.cuda.synchronize()
    for h in warm:
        aq.aq_destroy(h)

    # ---- epoch 0: first visits (uncompressed message), timed apart
    order0 = synth.epoch_order(cfg, 0)
    arena0, ids0 = gen_arena(0, order0), order0.cuda()
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        e0, e1 = ev(), ev()
        e0.record(stream)
        for s in range(steps_per_epoch):
            run_step(arena0, ids0, s, raw=True)
        e1.record(stream)
    torch.cuda.synchronize()
    first_ms = e0.elapsed_time(e1)
    aq.aq_configure(rcv, aq.AQ_RAW, None)
    first_bytes = cfg.n_samples * cfg.elems * ((4 + cfg.bits / 8 + 4 / cfg.group) + 6)
    if sweep:                                          # the steps of that epoch also carry the wires and the gradient kernels
        first_bytes += steps_per_epoch * (step_bytes - 2 * macro * cfg.elems * bpe)
    del arena0

    # ---- steady-state epochs: inputs resident in HBM before the clock starts
    arenas, id_lists = [], []
    for e in range(1, n_arenas + 1):
        order = synth.epoch_order(cfg, e)
        arenas.append(gen_arena(e, order))
        id_lists.append(order.cuda())
    torch.cuda.synchronize()
    del running

    def step_source(t):
        e = (t // steps_per_epoch) % n_arenas
        return arenas[e], id_lists[e], t % steps_per_epoch

    # ---- the timed region: `repeats` windows of exactly `steps` steps each
    graphs = None
    if use_graph:
        # one graph per step of a window (pointers differ from step to step); capture enqueues nothing
        graphs = []
        for t in range(steps):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                run_step(*step_source(warmup + t))
            graphs.append(g)
    windows_ms, walls_ms = [], []
    with torch.cuda.stream(stream):
        for t in range(warmup):
            graphs[t % steps].replay() if graphs else run_step(*step_source(t))
        torch.cuda.synchronize()
        with ClockSampler(local_rank) as clocks:
            repeats, r, t_next = 30, 0, warmup
            while r < repeats:
                t_begin, t_end = ev(), ev()
                if dist:
                    dist.barrier()
                torch.cuda.synchronize()
                wall0 = time.perf_counter()
                # about 0.1 ms of an idle-spinning kernel ahead of the start event: the host queues the event and the
                # first launches behind it, so that the clock starts with work waiting and not with launch latency
                if hasattr(torch.cuda, "_sleep"):
                    torch.cuda._sleep(200_000)
                t_begin.record(stream)
                for t in range(steps):
                    if graphs:
                        graphs[t].replay()
                    else:
                        run_step(*step_source(t_next + t), nxt=step_source(t_next + t + 1)[1:])
                t_end.record(stream)
                torch.cuda.synchronize()
                walls_ms.append((time.perf_counter() - wall0) * 1e3)
                if dist:
                    dist.barrier()
                torch.cuda.synchronize()
                # staged calls end with copies on the handles' own copy streams, which the event on `stream` does
                # not cover: there the window's time is the host's, taken between two whole-device synchronisations
                windows_ms.append(walls_ms[-1] if prefetching else t_begin.elapsed_time(t_end))
                t_next += steps
                r += 1
                if r == 3:                                        # size the run from the first windows
                    est = statistics.median(windows_ms)
                    want = max(30, math.ceil(args.min_timed_ms / max(est, 1e-3)))
                    if dist:                                      # the same count on every rank
                        t = torch.tensor([want], device="cuda")
                        dist.all_reduce(t, op=dist.ReduceOp.MAX)
                        want = int(t.item())
                    repeats = min(max(args.max_repeats, 30), want)
    total_steps = t_next
    # the slowest rank sets the time of every window
    if dist:
        t = torch.tensor(windows_ms, dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        windows_ms = t.cpu().tolist()
    elapsed_ms = statistics.median(windows_ms)

    staged_call_us = None
    if prefetching:
        # the calls' time once their rows have arrived: what stays on the critical path of a pipeline stage
        lat = []
        with torch.cuda.stream(stream):
            if ahead["key"] is not None:                      # use up the rows asked for by the last timed step
                run_step(*step_source(total_steps))
            for r in range(8):
                arena, ids_dev, sidx = step_source(total_steps + 1 + r)
                lo = sidx * macro
                prefetch(ids_dev, lo)
                torch.cuda.synchronize()
                a0, a1 = ev(), ev()
                a0.record(stream)
                aq.aq_encode(snd, arena[lo:lo + nb], ids_dev[lo:lo + nb], packed[:nb], scales[:nb])
                aq.aq_decode(rcv, packed[:nb], scales[:nb], ids_dev[lo:lo + nb], out[:nb])
                a1.record(stream)
                torch.cuda.synchronize()
                lat.append(a0.elapsed_time(a1) * 1e3)
        staged_call_us = statistics.median(lat)

    # ---- per-kernel durations: the steps that follow the timed ones, same handles, same data
    window = min(32, steps_per_epoch)
    with torch.cuda.stream(stream):
        passes = [kernel_pass(total_steps + 2 + r * window, window) for r in range(3)]
        grad_passes = [grad_pass(32) for r in range(3)] if sweep else None
    enc_ms = statistics.median(p[0] for p in passes)          # one disturbed pass must not move the figure
    dec_ms = statistics.median(p[1] for p in passes)

    # ---- the same steps with the two sides on streams of their own
    overlapped = None
    if not (hosted or use_graph or prefetching or stochastic or m_bits) and launches_per_step == 1:
        overlapped = two_stream_steps(aq, torch, snd, rcv, cfg, step_source, total_steps + 2 + 3 * window, macro, outs, stream,
                                      steps=max(steps, 32), reps=5)
        overlapped["GB/s"] = 2 * macro * cfg.elems * bpe / overlapped["ms_per_step"] / 1e6
        overlapped["frac_of_measured_hbm"] = overlapped["GB/s"] / measured_peak()[0]

    # ---- the same steps through the list forms: every sequence of the macro-batch named by a pointer of its own
    listed = None
    if overlapped is not None:
        listed = list_form_steps(aq, torch, snd, rcv, cfg, step_source, total_steps + 2 + 3 * window, macro, packed, scales, outs,
                                 stream, steps=max(steps, 32), reps=5)
        listed["GB/s"] = 2 * macro * cfg.elems * bpe / listed["ms_per_step"] / 1e6
        listed["frac_of_measured_hbm"] = listed["GB/s"] / measured_peak()[0]

    # ---- calls of the workload's own micro-batch size, enqueued back to back on the plain stream and as one CUDA graph
    micro = None
    if not (hosted or use_graph) and nb != cfg.n_batch:
        micro = micro_batch_calls(aq, torch, stream, snd, rcv, cfg, step_source, total_steps + 2 + 3 * window, macro, packed, scales, outs,
                                  bpe)
        for h in handles:
            aq.aq_configure(h, aq.AQ_BATCH, nb)

    status = aq.aq_status(snd) | aq.aq_status(rcv)
    digests_equal = aq.aq_state_checksum(snd) == aq.aq_state_checksum(rcv)
    assert status == 0 and digests_equal, "sender and receiver state diverged"

    peak, peak_kind = measured_peak()
    launch_bytes = nb * cfg.elems * bpe
    enc_gbs = launch_bytes / (enc_ms * 1e-3) / 1e9
    dec_gbs = launch_bytes / (dec_ms * 1e-3) / 1e9
    value = replicas.whole_job_rate(steps * step_bytes, world, elapsed_ms) / 1e9
    res = {
        "workload": label, "value": value, "ms_per_step": elapsed_ms / steps,
        "timed": {"windows": len(windows_ms), "steps_per_window": steps, "ms_per_step_min": min(windows_ms) / steps,
                  "ms_per_step_max": max(windows_ms) / steps, "gpu_ms_total": sum(windows_ms)},
        "samples_per_s": replicas.whole_job_rate(steps * macro, world, elapsed_ms),
        "frac_of_measured_hbm": value / world / peak, "frac_of_8000_spec": value / world / 8000.0,
        "step_bytes": step_bytes, "launch_bytes": launch_bytes, "bytes_per_element": bpe,
        "encode": {"achieved": enc_gbs, "frac": enc_gbs / peak, "avg_launch_ms": enc_ms},
        "decode": {"achieved": dec_gbs, "frac": dec_gbs / peak, "avg_launch_ms": dec_ms},
        "kernel_timing": f"CUDA events around {window * launches_per_step} back-to-back launches of the kernel, median of 3 passes right after the timed steps",
        "first_visit_epoch": {"ms": first_ms, "GB/s": first_bytes / (first_ms * 1e-3) / 1e9},
        "micro_batch_calls": micro, "two_streams": overlapped, "list_form": listed, "clocks": clocks.summary(),
        "gpu_launches_per_step": launches_per_step * (3 if sweep else 2) + (3 if sweep else 0),
        "peak": peak, "peak_kind": peak_kind,
        "shape": {"hidden": cfg.hidden, "seq": cfg.seq, "micro_batch": cfg.n_batch, "sequences_per_step": macro,
                  "sequences_per_launch": nb, "act_dtype": cfg.dtype, "bits": cfg.bits, "group": cfg.group,
                  "n_samples_per_side": cfg.n_samples, "steady_epochs_resident": n_arenas},
    }
    if sweep:
        q_ms = statistics.median(p[0] for p in grad_passes)
        d_ms = statistics.median(p[1] for p in grad_passes)
        res["quant_grad"] = {"bits": bbits, "achieved": grad_bytes / q_ms / 1e6, "frac": grad_bytes / q_ms / 1e6 / peak, "avg_launch_ms": q_ms}
        res["dequant_grad"] = {"bits": bbits, "achieved": grad_bytes / d_ms / 1e6, "frac": grad_bytes / d_ms / 1e6 / peak, "avg_launch_ms": d_ms}
    if staged_call_us is not None:
        res["staged_encode_plus_decode_us"] = staged_call_us
    if stage_cycles:
        res["stage_compute_ms_per_step"] = stage_ms

    if headline:
        if rank == 0 and not args.skip_aux:
            res["isolated_call"] = isolated_calls(aq, torch, stream, snd, rcv, cfg, arenas[0], id_lists[0])
            res["aux"] = aux_kernels(aq, torch, synth, stream, snd, cfg)
        # ---- end to end through the host-buffer entry points (pinned host memory both ways)
        res["e2e"] = None
        if not args.skip_e2e:
            res["e2e"] = run_e2e(aq, torch, cfg, snd, rcv, arenas[0], id_lists[0], args.e2e_steps, dist, macro, bpe)
        res["cpu_baseline"] = None
        if rank == 0 and not args.skip_cpu:
            gbs, sps, n, secs = time_oracle(cfg, args.cpu_seconds, "cuda")
            res["cpu_baseline"] = {
                "value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "samples_per_s": sps,
                "sample": f"steady-state encode+decode of {n} whole sequences ({n * cfg.elems} elements, {secs:.1f} s), single thread",
                "all_cores": time_oracle_all_cores(cfg, args.cpu_seconds, "cuda")}
    res["cfg"] = cfg
    for h in handles:
        aq.aq_destroy(h)
    del arenas, id_lists, packed, scales, out, outs
    torch.cuda.empty_cache()
    return res


def measure_pipeline(args, env):
    """One boundary per pair of ranks: rank 2p owns the sender handle and the activations, rank 2p+1 the
    receiver handle; codes, steps and (epoch 0) the raw blocks cross between the two GPUs through
    BoundaryLink (NCCL send / recv into the receiver's own buffers), after which aq_decode reads locally.
    Timed like the replica run: windows of `steps` steps between barriers, the slowest rank sets the time."""
    import torch
    import paper_2206_01299_b200 as aq
    from paper_2206_01299_b200.link import BoundaryLink
    from fixtures import replicas, synth

    rank, world, dist, stream = env.rank, env.world, env.dist, env.stream
    assert dist is not None and world % 2 == 0, "--topology pipeline needs an even number of ranks"
    pair, sender = rank // 2, rank % 2 == 0
    recipe, macro, label = WORKLOADS[args.workload]
    cfg = getattr(synth, recipe)
    if args.n_samples:
        cfg = synth.shrink(cfg, args.n_samples)
    cfg = replicas.shard_for_rank(cfg, pair, world // 2)
    nb, steps, warmup = macro, args.steps, args.warmup
    steps_per_epoch = cfg.n_samples // macro
    bpe = bytes_per_element(cfg.bits, cfg.group)

    h = aq.aq_create(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group)
    aq.aq_configure(h, aq.AQ_DTYPE, aq.AQ_FP16 if cfg.dtype == "fp16" else aq.AQ_BF16)
    aq.aq_configure(h, aq.AQ_BATCH, nb)
    aq.aq_configure(h, aq.AQ_STREAM, stream.cuda_stream)
    first = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    aq.aq_configure(h, aq.AQ_FIRST_FLAGS, first)
    wire_dev = "cuda" if args.backend == "nccl" else "cpu"       # gloo moves host memory only
    link = BoundaryLink(dist, rank + 1 if sender else rank - 1, nb, cfg.packed_bytes, cfg.groups, cfg.elems, cfg.torch_dtype, wire_dev)
    packed = torch.empty((nb, cfg.packed_bytes), dtype=torch.uint8, device="cuda")
    scales = torch.empty((nb, cfg.groups), dtype=torch.float32, device="cuda")
    out = torch.empty((nb, cfg.seq, cfg.hidden), dtype=cfg.torch_dtype, device="cuda")
    orders = [synth.epoch_order(cfg, e) for e in range(2)]

    def arena_of(epoch):
        a = torch.empty((cfg.n_samples, cfg.seq, cfg.hidden), dtype=cfg.torch_dtype, device="cuda")
        for c in range(0, cfg.n_samples, 16):
            a[c:c + 16] = synth.activation(cfg, orders[epoch][c:c + 16], epoch, device="cuda")
        return a

    def step(epoch, arena, s):
        ids = orders[epoch][s * macro:(s + 1) * macro]
        with torch.cuda.stream(stream):
            if sender:
                act = arena[s * macro:(s + 1) * macro]
                aq.aq_encode(h, act, ids.cuda(), packed, scales)
                stream.synchronize()                      # the link's sends run on the process group's stream
                link.send(ids, first, packed, scales, act)
            else:
                _, _, p, sc, raw = link.recv(expect_ids=ids)
                if wire_dev == "cpu":
                    p, sc, raw = p.cuda(), sc.cuda(), (None if raw is None else raw.cuda())
                aq.aq_configure(h, aq.AQ_RAW, raw)
                aq.aq_decode(h, p, sc, ids.cuda(), out)
                stream.synchronize()

    arena = arena_of(0) if sender else None
    for s in range(steps_per_epoch):                       # epoch 0: first visits, untimed
        step(0, arena, s)
    arena = arena_of(1) if sender else None
    windows_ms, t = [], 0
    for s in range(warmup):
        step(1, arena, (t := t + 1) % steps_per_epoch)
    for r in range(30):
        dist.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for s in range(steps):
            step(1, arena, (t := t + 1) % steps_per_epoch)
        torch.cuda.synchronize()
        windows_ms.append((time.perf_counter() - t0) * 1e3)
    ms = torch.tensor(windows_ms, dtype=torch.float64, device=wire_dev)
    dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    digest = torch.tensor([aq.aq_state_checksum(h) & 0x7FFFFFFFFFFFFFFF], dtype=torch.int64, device=wire_dev)
    both = [torch.zeros_like(digest) for _ in range(world)]
    dist.all_gather(both, digest)
    assert all(both[2 * p].item() == both[2 * p + 1].item() for p in range(world // 2)), "sender and receiver state diverged"
    assert aq.aq_status(h) == 0
    aq.aq_destroy(h)
    elapsed = statistics.median(ms.cpu().tolist())
    step_bytes = 2 * macro * cfg.elems * bpe
    value = (world // 2) * steps * step_bytes / (elapsed * 1e-3) / 1e9
    wire = macro * (cfg.packed_bytes + cfg.groups * 4) + 4 * (1 + 2 * macro)
    return {"metric": "activation encode+decode GB/s", "value": value, "unit": "GB/s", "n_gpus": world, "steps": steps,
            "warmup": warmup, "ms_per_step": elapsed / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": label, "topology": f"pipeline: {world // 2} boundaries, sender and receiver of each on two GPUs, "
                       "message over torch.distributed send/recv", "sequences_per_step": macro, "wire_bytes_per_step": wire,
                       "timing": "host clock between barriers, median of 30 windows, slowest rank"},
            "gpu_launches": 30 * steps}


def two_stream_steps(aq, torch, snd, rcv, cfg, step_source, first_step, macro, outs, home_stream, steps, reps):
    """Encode and decode of consecutive steps on two streams, the way two stages on two devices work: the
    receiver decodes message t while the sender already encodes message t+1 (two wire buffers; events hand
    a buffer from one stream to the other and back).  The forward codec only (no wire copy, no gradients),
    same handles and data as the timed steps; median of `reps` runs of `steps` steps, by events."""
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    wires = [(torch.empty((macro, cfg.packed_bytes), dtype=torch.uint8, device="cuda"),
              torch.empty((macro, cfg.groups), dtype=torch.float32, device="cuda")) for _ in range(2)]
    torch.cuda.synchronize()
    aq.aq_configure(snd, aq.AQ_STREAM, sa.cuda_stream)
    aq.aq_configure(rcv, aq.AQ_STREAM, sb.cuda_stream)
    times, t0 = [], first_step
    for rep in range(reps + 1):
        enc_done = [torch.cuda.Event() for _ in range(steps)]
        dec_done = [torch.cuda.Event() for _ in range(steps)]
        begin, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        if hasattr(torch.cuda, "_sleep"):
            with torch.cuda.stream(sa):
                torch.cuda._sleep(400_000)                # work queued on both streams before the clock starts
        begin.record(sa)
        sb.wait_event(begin)
        for t in range(steps):
            arena, ids_dev, s = step_source(t0 + t)
            lo = s * macro
            p, sc = wires[t % 2]
            if t >= 2:
                sa.wait_event(dec_done[t - 2])            # the receiver has read this wire buffer
            aq.aq_encode(snd, arena[lo:lo + macro], ids_dev[lo:lo + macro], p, sc)
            enc_done[t].record(sa)
            sb.wait_event(enc_done[t])
            aq.aq_decode(rcv, p, sc, ids_dev[lo:lo + macro], outs[t % len(outs)])
            dec_done[t].record(sb)
        end.record(sb)
        torch.cuda.synchronize()
        if rep:                                           # the first run warms the streams up
            times.append(begin.elapsed_time(end) / steps)
        t0 += steps
    aq.aq_configure(snd, aq.AQ_STREAM, home_stream.cuda_stream)
    aq.aq_configure(rcv, aq.AQ_STREAM, home_stream.cuda_stream)
    return {"ms_per_step": statistics.median(times), "steps": steps, "runs": reps,
            "note": "sender and receiver handles on two streams, two wire buffers: decode of step t beside encode of step t+1"}


def list_form_steps(aq, torch, snd, rcv, cfg, step_source, first_step, macro, packed, scales, outs, stream, steps, reps):
    """The timed step through aq_encode_list / aq_decode_list: the macro-batch's sequences are handed over as
    `macro` separate buffers (here: the rows of the arena and of the wire and output buffers, each named by its
    own pointer), one launch per side.  Same stream, same data as the timed steps; median of `reps` runs."""
    row = lambda t: torch.tensor([t[y].data_ptr() for y in range(macro)], dtype=torch.int64, device="cuda")
    packed_l, scales_l = row(packed), row(scales)
    outs_l = [row(o) for o in outs]
    acts_l = {}
    for t in range(steps):                                   # pointer arrays of the steps, built before the clock starts
        arena, ids_dev, s = step_source(first_step + t)
        key = (arena.data_ptr(), s)
        if key not in acts_l:
            acts_l[key] = row(arena[s * macro:(s + 1) * macro])
    torch.cuda.synchronize()
    times = []
    with torch.cuda.stream(stream):
        for rep in range(reps + 1):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if hasattr(torch.cuda, "_sleep"):
                torch.cuda._sleep(400_000)
            a.record(stream)
            for t in range(steps):
                arena, ids_dev, s = step_source(first_step + t)
                ids = ids_dev[s * macro:(s + 1) * macro]
                aq.aq_encode_list(snd, acts_l[(arena.data_ptr(), s)], ids, packed_l, scales_l)
                aq.aq_decode_list(rcv, packed_l, scales_l, ids, outs_l[t % len(outs_l)])
            b.record(stream)
            torch.cuda.synchronize()
            if rep:
                times.append(a.elapsed_time(b) / steps)
    return {"ms_per_step": statistics.median(times), "steps": steps, "runs": reps,
            "note": "aq_encode_list + aq_decode_list, one pointer per sequence of the macro-batch"}


def micro_batch_calls(aq, torch, stream, snd, rcv, cfg, step_source, first_step, macro, packed, scales, outs, bpe, steps=24):
    """Sustained throughput of calls the size of the workload's own micro-batch (1 or 8 sequences): the
    micro-batches of `steps` macro-batches, each encoded then decoded, enqueued back to back -- once call by
    call through the binding on the plain stream, once as CUDA graphs of one macro-batch each."""
    nb = cfg.n_batch
    for h in (snd, rcv):
        aq.aq_configure(h, aq.AQ_BATCH, nb)
    per_step = macro // nb
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def one_step(t):
        arena, ids_dev, s = step_source(t)
        for l in range(per_step):
            lo = s * macro + l * nb
            aq.aq_encode(snd, arena[lo:lo + nb], ids_dev[lo:lo + nb], packed[l * nb:(l + 1) * nb], scales[l * nb:(l + 1) * nb])
            aq.aq_decode(rcv, packed[l * nb:(l + 1) * nb], scales[l * nb:(l + 1) * nb], ids_dev[lo:lo + nb],
                         outs[t % len(outs)][l * nb:(l + 1) * nb])

    with torch.cuda.stream(stream):
        one_step(first_step)
        torch.cuda.synchronize()
        a, b = ev(), ev()
        if hasattr(torch.cuda, "_sleep"):
            torch.cuda._sleep(2_000_000)                  # a millisecond of queued work ahead of the clock
        a.record(stream)
        for t in range(steps):
            one_step(first_step + 1 + t)
        b.record(stream)
        torch.cuda.synchronize()
        ms_stream = a.elapsed_time(b)
        graphs = []
        for t in range(steps):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                one_step(first_step + 1 + steps + t)
            graphs.append(g)
        graphs[0].replay()
        torch.cuda.synchronize()
        a, b = ev(), ev()
        a.record(stream)
        for g in graphs:
            g.replay()
        b.record(stream)
        torch.cuda.synchronize()
        ms_graph = a.elapsed_time(b)
    calls = steps * per_step                              # encode + decode pairs
    pair_bytes = 2 * nb * cfg.elems * bpe
    return {"sequences_per_call": nb, "calls": 2 * calls,
            "stream": {"us_per_call": ms_stream * 1e3 / (2 * calls), "GB/s": calls * pair_bytes / ms_stream / 1e6},
            "graph": {"us_per_call": ms_graph * 1e3 / (2 * calls), "GB/s": calls * pair_bytes / ms_graph / 1e6},
            "note": "encode then decode of every micro-batch, back to back on one stream; us_per_call counts each encode and each decode"}


def isolated_calls(aq, torch, stream, snd, rcv, cfg, arena, ids_dev, reps=40):
    """Latency of one micro-batch call (the workload's own micro-batch size) on an idle GPU: the call
    is captured once into a CUDA graph, so that the figure is the GPU's and not the Python binding's;
    each replay runs between two events on the otherwise empty stream; median over `reps` replays."""
    nb = cfg.n_batch
    for h in (snd, rcv):
        aq.aq_configure(h, aq.AQ_BATCH, nb)
    packed = torch.empty((nb, cfg.packed_bytes), dtype=torch.uint8, device="cuda")
    scales = torch.empty((nb, cfg.groups), dtype=torch.float32, device="cuda")
    out = torch.empty((nb, cfg.seq, cfg.hidden), dtype=cfg.torch_dtype, device="cuda")
    slots = [(r * 37 % (cfg.n_samples // nb)) * nb for r in range(8)]
    graphs = []
    torch.cuda.synchronize()
    for lo in slots:
        ge, gd = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        with torch.cuda.graph(ge, stream=stream):
            aq.aq_encode(snd, arena[lo:lo + nb], ids_dev[lo:lo + nb], packed, scales)
        with torch.cuda.graph(gd, stream=stream):
            aq.aq_decode(rcv, packed, scales, ids_dev[lo:lo + nb], out)
        graphs.append((ge, gd))
    enc, dec = [], []
    with torch.cuda.stream(stream):
        for r in range(reps + 8):
            ge, gd = graphs[r % len(graphs)]
            e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            e[0].record(stream)
            ge.replay()
            e[1].record(stream)
            torch.cuda.synchronize()
            e[2].record(stream)
            gd.replay()
            e[3].record(stream)
            torch.cuda.synchronize()
            if r >= 8:
                enc.append(e[0].elapsed_time(e[1]) * 1e3)
                dec.append(e[2].elapsed_time(e[3]) * 1e3)
    bytes_call = nb * cfg.elems * bytes_per_element(cfg.bits, cfg.group)
    enc_us, dec_us = statistics.median(enc), statistics.median(dec)
    return {"sequences_per_call": nb, "encode_us": enc_us, "decode_us": dec_us,
            "encode_GB/s": bytes_call / enc_us / 1e3, "decode_GB/s": bytes_call / dec_us / 1e3}


def aux_kernels(aq, torch, synth, stream, h, cfg):
    """The remaining kernels of the path, each timed alone over rotating buffers larger than L2:
    gradient quantize / dequantize (the 'Backward path' workload: 4 x 1024 x 1600 per call, and the
    same kernels on 16 such micro-batches handed over in one call) and the state digest.
    Per call: CUDA events around 60 calls issued back to back through the binding ("stream"), and
    around 5 replays of a CUDA graph of 12 calls ("graph": no host pacing between the launches)."""
    from dataclasses import replace
    g = synth.BACKWARD
    res = {}
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def timed(fn, reps):
        a, b = ev(), ev()
        a.record(stream)
        for _ in range(reps):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b)

    with torch.cuda.stream(stream):
        for label, gw, sets in (("", g, 12), ("_x16", replace(g, n_batch=16 * g.n_batch), 3)):
            n = gw.elems
            grads = [synth.gradient(gw, i, device="cuda") for i in range(sets)]          # sets x n x 2 B > L2
            for bits in g.bits:
                packed = [torch.empty(n * bits // 8, dtype=torch.uint8, device="cuda") for _ in range(sets)]
                scales = [torch.empty(n // g.group, dtype=torch.float32, device="cuda") for _ in range(sets)]
                outs = [torch.empty(n, dtype=torch.float16, device="cuda") for _ in range(sets)]
                for name in ("quant", "dequant"):
                    def sweep():
                        for i in range(sets):
                            if name == "quant":
                                aq.aq_quant_grad(h, grads[i], n, bits, packed[i], scales[i])
                            else:
                                aq.aq_dequant_grad(h, packed[i], scales[i], n, bits, outs[i])
                    sweep()
                    torch.cuda.synchronize()
                    ms_stream = timed(sweep, 5) / (5 * sets)
                    graph = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(graph, stream=stream):
                        sweep()
                    graph.replay()
                    torch.cuda.synchronize()
                    ms_graph = timed(graph.replay, 5) / (5 * sets)
                    ms = min(ms_stream, ms_graph)
                    res[f"{name}_grad_b{bits}{label}"] = {
                        "ms": ms, "ms_stream": ms_stream, "ms_graph": ms_graph,
                        "GB/s": n * (2 + bits / 8 + 4 / g.group) / (ms * 1e-3) / 1e9}
            del grads
    t0 = time.perf_counter()
    aq.aq_state_checksum(h)
    dt = time.perf_counter() - t0
    res["state_checksum"] = {"ms": dt * 1e3, "GB/s": cfg.n_samples * cfg.elems * 2 / dt / 1e9}
    return res


def run_e2e(aq, torch, cfg, snd, rcv, arena, ids_dev, steps, dist, macro, bpe):
    """The step through the host-buffer calls: activations start in pinned host memory, codes and
    scales cross to pinned host memory and back (the wire), the reconstructed activation ends in
    pinned host memory.  Uses the handles of the device-resident run (every sample already seen),
    so every timed visit is a steady-state delta visit."""
    from fixtures import replicas
    nb = macro
    for h in (snd, rcv):
        aq.aq_configure(h, aq.AQ_BATCH, nb)
    ids = ids_dev.cpu()
    n_sets = min(steps, 4)
    acts = [arena[s * nb:(s + 1) * nb].cpu().pin_memory() for s in range(n_sets)]
    # two wire buffers: the receiver reads message t while the sender writes message t+1
    packed = [torch.empty((nb, cfg.packed_bytes), dtype=torch.uint8).pin_memory() for _ in range(2)]
    scales = [torch.empty((nb, cfg.groups), dtype=torch.float32).pin_memory() for _ in range(2)]
    out = torch.empty_like(acts[0]).pin_memory()
    # the receiving side gets a stream of its own, so that its device-to-host copy of step t and
    # the sender's host-to-device copy of step t+1 use the two directions of the link together
    rcv_stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    aq.aq_configure(rcv, aq.AQ_STREAM, rcv_stream.cuda_stream)
    id_sets = [ids[s * nb:(s + 1) * nb].contiguous() for s in range(n_sets)]

    def send(t):
        aq.aq_encode_host(snd, acts[t % n_sets], id_sets[t % n_sets], packed[t % 2], scales[t % 2])

    def receive(t):
        aq.aq_decode_host(rcv, packed[t % 2], scales[t % 2], None, id_sets[t % n_sets], out)

    def run_serial(k):
        for t in range(k):
            send(t)
            receive(t)

    def run_pipelined(k):
        # the sender's calls in this thread, the receiver's in a second one (the calls release the GIL);
        # a wire buffer goes back to the sender when the receiver has read it
        ready = [threading.Semaphore(0) for _ in range(2)]
        free = [threading.Semaphore(1) for _ in range(2)]
        failed = []

        def receiver():
            try:
                for t in range(k):
                    ready[t % 2].acquire()
                    receive(t)
                    free[t % 2].release()
            except Exception as e:                            # let the sender finish, report afterwards
                failed.append(e)
                for f in free:
                    f.release()

        th = threading.Thread(target=receiver)
        th.start()
        for t in range(k):
            free[t % 2].acquire()
            send(t)
            ready[t % 2].release()
        th.join()
        if failed:
            raise failed[0]

    def timed(fn):
        fn(3)                                                 # warm-up; the first call allocates the staging buffers
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        t0 = time.perf_counter()
        fn(steps)
        torch.cuda.synchronize()
        return time.perf_counter() - t0

    dt_serial = timed(run_serial)
    dt = timed(run_pipelined)
    dt = replicas.max_over_ranks(dt, dist, "cuda")
    assert aq.aq_status(snd) == 0 and aq.aq_status(rcv) == 0
    assert aq.aq_state_checksum(snd) == aq.aq_state_checksum(rcv)
    world = dist.get_world_size() if dist else 1
    act_b = nb * cfg.elems * 2
    wire_b = nb * (cfg.packed_bytes + cfg.groups * 4)
    step_bytes = 2 * nb * cfg.elems * bpe
    return {"value": world * steps * step_bytes / dt / 1e9, "unit": "GB/s", "ms_per_step": dt / steps * 1e3,
            "h2d_bytes_per_step": act_b + wire_b + 2 * nb * 4, "d2h_bytes_per_step": wire_b + act_b,
            "steps": steps, "serial_ms_per_step": dt_serial / steps * 1e3,
            "note": "aq_encode_host + aq_decode_host on pinned host buffers, host clock; the receiver's calls run in a "
                    "second host thread and stream beside the sender's, two wire buffers between them "
                    "(serial_ms_per_step: the two calls one after the other)"}


def main():
    args = parse_args()
    if args.kernel_hash:
        print(kernel_source_hash())
        return
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        if rank == 0:
            from fixtures import synth
            cfg = getattr(synth, WORKLOADS[args.workload][0])
            if args.n_samples:
                cfg = synth.shrink(cfg, args.n_samples)
            run_reference(args, cfg)
        return

    import torch
    import paper_2206_01299_b200 as aq
    aq.lib()                                         # fails loudly when the CUDA library is missing
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU path"
    local_rank = local_rank % torch.cuda.device_count() if args.backend == "gloo" else local_rank
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        if args.backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        else:
            dist.init_process_group("gloo")
    if args.prefetch and not args.hosted:
        raise SystemExit("--prefetch needs --hosted")
    if args.hosted and args.m_bits == 32:
        raise SystemExit("the binary32 store is not offered in host memory")
    env = Env(rank, local_rank, world, dist, torch.cuda.Stream())

    if args.topology == "pipeline":
        line = measure_pipeline(args, env)
        dist.destroy_process_group()
        if rank == 0:
            print(json.dumps(line))
        return

    head = measure_boundary(args, env, args.workload, args.steps, args.warmup, headline=True)
    plain = (args.rounding == "interval" and not args.m_bits and not args.hosted and not args.per_launch and not args.graph
             and not args.n_samples)
    others = {}
    which = args.configs or ("all" if world == 1 and plain else "headline")
    if which == "all" and world == 1:
        for name in WORKLOADS:
            if name != args.workload:
                r = measure_boundary(args, env, name, args.steps, args.warmup, headline=False)
                r.pop("cfg")
                others[name] = r
    if dist:
        dist.destroy_process_group()
    if rank != 0:
        return

    cfg = head.pop("cfg")
    sh = head["shape"]
    traffic = None
    rec = NCU_TRAFFIC.get(args.workload)
    if rec and plain and rec["kernel_hash"] == kernel_source_hash():
        traffic = rec["encode_bytes_per_element"] * sh["sequences_per_launch"] * cfg.elems
    m_state = cfg.n_samples * (cfg.elems * 2 if not args.m_bits else cfg.elems * args.m_bits // 8 + (0 if args.m_bits == 32 else cfg.groups * 4))
    line = {
        "metric": "activation encode+decode GB/s", "value": head["value"], "unit": "GB/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": head["workload"], "hidden": cfg.hidden, "seq": cfg.seq,
                   "micro_batch": cfg.n_batch, "sequences_per_step": sh["sequences_per_step"],
                   "sequences_per_launch": sh["sequences_per_launch"],
                   "launch_shape": (f"one aq_encode / aq_decode call per {sh['sequences_per_launch']} sequences (the macro-batch of "
                                    f"{sh['sequences_per_step']} micro-batches of {cfg.n_batch}); calls of one micro-batch are under micro_batch_calls"),
                   "cuda_graph": bool(args.graph), "rounding": args.rounding, "m_bits": args.m_bits or 16,
                   "m_in": ("host memory (page-locked), staged through HBM by aq_prefetch, written back on a copy stream; step time by the host clock" if args.prefetch
                            else "host memory (page-locked, mapped)" if args.hosted else "HBM"),
                   "act_dtype": cfg.dtype, "bits": cfg.bits, "group": cfg.group, "n_samples_per_side": cfg.n_samples,
                   "m_bytes_per_side": m_state, "steady_epochs_resident": sh["steady_epochs_resident"],
                   "l2": f"inputs larger than L2 (each step touches {int(sh['sequences_per_step'] * cfg.elems * 6 / 1e6)} MB of fresh HBM; no flush needed)",
                   "parallelism": f"dp{world} replicas, no collective"},
        "timed": head["timed"],
        # step time x median sampled SM clock: compares runs taken at different clocks under the power cap
        "sm_kcycles_per_step": (head["ms_per_step"] * head["clocks"]["sm_mhz"] if head["clocks"]["sm_mhz"] else None),
        "samples_per_s": head["samples_per_s"],
        "frac_of_measured_hbm": head["frac_of_measured_hbm"], "frac_of_8000_spec": head["frac_of_8000_spec"],
        "roofline": {"bound": "hbm", "kernel": "encode_kernel", "achieved": head["encode"]["achieved"], "peak": head["peak"], "unit": "GB/s",
                     "frac": head["encode"]["frac"], "peak_kind": head["peak_kind"],
                     "traffic": traffic, "traffic_from": (rec or {}).get("capture"),
                     "algorithmic_bytes_per_launch": head["launch_bytes"], "avg_launch_ms": head["encode"]["avg_launch_ms"],
                     "timing": head["kernel_timing"],
                     "decode_kernel": head["decode"]},
        "first_visit_epoch": head["first_visit_epoch"],
        "micro_batch_calls": head["micro_batch_calls"], "two_streams": head.get("two_streams"), "list_form": head.get("list_form"),
        "e2e": head.get("e2e"), "cpu_baseline": head.get("cpu_baseline"),
        "gpu_launches": args.steps * head["gpu_launches_per_step"] * head["timed"]["windows"],
        "clocks": head["clocks"],
    }
    for k in ("quant_grad", "dequant_grad", "staged_encode_plus_decode_us", "stage_compute_ms_per_step", "isolated_call", "aux"):
        if k in head:
            line[k] = head[k]
    if others:
        line["configs"] = others
    if "aux" in head:
        line.setdefault("configs", {})["backward"] = {
            "workload": "Backward path (configs[3]): 4 x 1024 x 1600 fp16 gradients per call, 8 and 4 bit, group 64; _x16 = 16 such micro-batches in one call",
            **{k: v for k, v in head["aux"].items() if k != "state_checksum"}}
    print(json.dumps(line))


if __name__ == "__main__":
    main()
