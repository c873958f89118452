#!/usr/bin/env python3
"""Throughput of the Tetra decode-and-multiply path on B200.

A step is one batch-1 weight pass over every projection matrix of a
Qwen3-8B-shaped model (252 matrices, about 1.8 GB of 48-bit words, tails,
scales, activations and results) on synthetic seeded inputs.  The metric is the
rate at which those algorithmic bytes are consumed (GB/s); the roofline is the
same bytes over the measured HBM copy bandwidth.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--model qwen3-8b] [--impl ours|reference]

One JSON line on stdout (rank 0).  Under torchrun every rank runs an
independent replica of the pass on its own GPU (weak scaling, no collective on
the data path); the time is the maximum over ranks.
"""
import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "tetra_gemv_batch1_hbm_gbps"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes per algorithmic byte of k_gemv_units, from the ncu capture summarised in
# profiles/k_gemv_units_qwen3_8b.md (dram__bytes_read.sum + dram__bytes_write.sum = 202.5 MB
# for the 198.4 MB of the first 4 layers; every code byte is read once, so traffic grows in
# proportion to the matrices read and the full pass is scaled by its byte count).
TRAFFIC_PER_ALGORITHMIC_BYTE = 1.02
# Warp-instructions of k_gemv_units per 32 blocks (one block per lane), by pipe, and wavefronts of the
# shared-memory/L1 data pipe, from the same capture (smsp__inst_executed.sum and
# sm__inst_executed_pipe_{alu,fmaheavy,lsu}.sum over the blocks processed / 32).
KERNEL_COUNTERS = {"instr": 85.9, "alu": 40.1, "fmaheavy": 32.0, "lsu": 9.6, "wavefronts": 21.0}


def issue_bound_gbs(sm_mhz, sms=148):
    """Rate at which the kernel would consume code bytes if every issue slot were used: four schedulers
    per SM, one warp-instruction per cycle each, KERNEL_COUNTERS['instr'] per 32 blocks of 6 bytes."""
    return sms * 4 * sm_mhz * 1e6 / KERNEL_COUNTERS["instr"] * 32 * 6 / 1e9


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------
# clocks during the timed region (read-only NVML queries)
# --------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, index):
        self.samples, self.reasons, self.power = [], set(), []
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                for bit, name in self.REASONS.items():
                    if mask & bit and name != "gpu_idle":
                        self.reasons.add(name)
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
            except Exception:
                pass
            time.sleep(0.02)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "power_w_max": max(self.power) if self.power else None, "samples": len(self.samples)}


# --------------------------------------------------------------------------
def timed(torch, fn, steps, warmup, stream):
    """Average milliseconds per call of fn, CUDA events on the launching stream."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        fn()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def oracle_sample(dp, orc, layers, threads, compare_with=None):
    """Times the CPU oracle on the first `layers` layers' matrices of the pass.
    Returns (seconds, bytes processed, worst ratio to the tolerance)."""
    from oracle.check import ABS_COEF, ABS_FLOOR, oracle_product
    per_layer = 7
    items = list(range(min(len(dp.items), layers * per_layer)))
    inputs = [dp.host_inputs(i) for i in items]
    t0 = time.perf_counter()
    refs = [oracle_product(orc, m, dp.gain, threads=threads) for m in inputs]
    dt = time.perf_counter() - t0
    nbytes = sum(dp.items[i]["bytes"] for i in items)
    worst = None
    if compare_with is not None:
        worst = 0.0
        for i, ref in zip(items, refs):
            it = dp.items[i]
            y = compare_with[it["yoff"]:it["yoff"] + it["N"]].astype(np.float64)
            bound = ABS_COEF * ref["termnorm"] + ABS_FLOOR
            worst = max(worst, float(np.max(np.abs(y - ref["y"]) / bound)))
    return dt, nbytes, worst, len(items)


def run_reference(args, rank, world):
    """The oracle as it stands, on the host cores (rank 0 only)."""
    if rank != 0:
        return
    import oracle
    from paper_2609_35465_b200 import shapes, synth
    from oracle.check import make_matrix, oracle_product
    orc = oracle.get()
    model = shapes.MODELS[args.model]
    mats = model.layer_matrices()               # one layer per step: a bounded sample of the pass
    inputs = [make_matrix(args.seed, i, m.N, m.K, True) for i, m in enumerate(mats)]
    nbytes = sum(m.N * (m.blocks * 6 + m.ntail * 2 + 8) + m.K * 2 for m in mats)
    threads = os.cpu_count() or 1
    for _ in range(args.warmup):
        [oracle_product(orc, m, synth.DEFAULT_GAIN, threads=threads) for m in inputs]
    t0 = time.perf_counter()
    for _ in range(args.steps):
        [oracle_product(orc, m, synth.DEFAULT_GAIN, threads=threads) for m in inputs]
    dt = (time.perf_counter() - t0) / args.steps
    value = nbytes / dt / 1e9
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s batch-1 weight pass; each step is one layer (7 of %d matrices)"
                               % (model.name, 7 * model.layers)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": "one layer (7 matrices, %d bytes) per step" % nbytes},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--model", default="qwen3-8b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--layers", type=int, default=0, help="use only the first L layers (profiling runs)")
    ap.add_argument("--no-extras", action="store_true", help="skip the secondary arms and the CPU baseline")
    ap.add_argument("--batched-only", type=int, default=0, metavar="VECTORS",
                    help="profiling runs: two rounds of tetra_gemv_batched over 12 copies of the 4096 x 12288 "
                         "matrix with this many vectors, nothing else, no JSON line")
    ap.add_argument("--encode-only", type=int, default=0, metavar="BLOCKS",
                    help="profiling runs: two tetra_encode_blocks launches on this many Gaussian blocks, nothing else, "
                         "no JSON line")
    ap.add_argument("--list-only", type=int, default=0, metavar="LAYERS",
                    help="profiling runs: the dependency steps of this many layers (q,k,v | o | gate,up | down), one "
                         "tetra_gemv_list launch each, three rounds, nothing else, no JSON line")
    ap.add_argument("--q4-list-only", type=int, default=0, metavar="LAYERS",
                    help="profiling runs: three tetra_q4_list_run passes over the v, o and down shapes of this many "
                         "layers (groups of 128), nothing else, no JSON line")
    ap.add_argument("--q4-only", default="", metavar="N,K,G,BATCH",
                    help="profiling runs: three tetra_q4_gemv launches on one synthetic matrix, nothing else, "
                         "no JSON line")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_2609_35465_b200 import ranks, shapes
    from paper_2609_35465_b200 import build as tbuild
    from paper_2609_35465_b200.workload import DevicePass
    from paper_2609_35465_b200 import tetra as tetra_mod

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    if rank == 0 and not os.environ.get("TETRA_LIB"):
        tbuild.build()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    elif not os.path.exists(tbuild.LIB) and not os.environ.get("TETRA_LIB"):
        tbuild.build()

    if args.encode_only:
        from paper_2609_35465_b200 import synth, tetra
        ne = args.encode_only
        wd = torch.from_numpy(synth.normal(11, 0, 20, ne * 24).reshape(ne, 24).astype(np.float32)).cuda()
        enc_table = tetra.tetra_build_table(synth.DEFAULT_GAIN)
        for _ in range(2):
            tetra.tetra_encode_blocks(wd, enc_table)
        torch.cuda.synchronize()
        return
    if args.q4_list_only:
        from paper_2609_35465_b200 import synth, tetra
        mdl = shapes.MODELS[args.model]
        kv_dim, q_dim = mdl.kv_heads * mdl.head_dim, mdl.q_heads * mdl.head_dim
        qitems = []
        for layer in range(args.q4_list_only):
            for qN, qK in ((kv_dim, mdl.hidden), (mdl.hidden, q_dim), (mdl.hidden, mdl.intermediate)):
                qn = torch.from_numpy(synth.q4_nibbles(args.seed + 17, qN, min(qN, 4096), qK)).cuda()
                sc, of = synth.q4_scales_offsets(args.seed + 17, qN, qN, qK // 128)
                qitems.append(dict(packed=tetra.tetra_q4_pack(qn, torch.from_numpy(sc).cuda(), torch.from_numpy(of).cuda(),
                                                              qN, qK, 128), N=qN, K=qK,
                                   x=torch.from_numpy(synth.activations(args.seed + 17, layer, qK, 1)[0]).cuda(),
                                   y=torch.empty(qN, dtype=torch.float32, device="cuda")))
        qws = tetra.tetra_q4_list_plan(tetra.make_q4_problems(qitems), 128)
        for _ in range(3):
            tetra.tetra_q4_list_run(qws, 128)
        torch.cuda.synchronize()
        return
    if args.q4_only:
        from paper_2609_35465_b200 import synth, tetra
        qN, qK, qG, qB = (int(v) for v in args.q4_only.split(","))
        rows_src = min(qN, 4096)
        qn = torch.from_numpy(synth.q4_nibbles(args.seed + 17, qN, rows_src, qK)).cuda()
        qn = qn.repeat((qN + rows_src - 1) // rows_src, 1)[:qN].contiguous()
        sc, of = synth.q4_scales_offsets(args.seed + 17, qN, qN, qK // qG)
        pk = tetra.tetra_q4_pack(qn, torch.from_numpy(sc).cuda(), torch.from_numpy(of).cuda(), qN, qK, qG)
        xq = torch.from_numpy(synth.activations(args.seed + 17, 1, qK, qB)).cuda()
        yq = torch.empty((qB, qN), dtype=torch.float32, device="cuda")
        for _ in range(3):
            tetra.tetra_q4_gemv(pk, xq, yq, qN, qK, qG, qB)
        torch.cuda.synchronize()
        return
    if args.list_only:
        from paper_2609_35465_b200 import tetra
        lp = DevicePass(shapes.MODELS[args.model].all_matrices()[:7 * args.list_only], seed=args.seed + 5)
        lists = [tetra.make_problems(lp.items[lo + a:lo + b]) for lo in range(0, len(lp.items), 7)
                 for a, b in ((0, 3), (3, 4), (4, 6), (6, 7))]
        for _ in range(3):
            for pr in lists:
                tetra.tetra_gemv_list(pr, lp.table)
        torch.cuda.synchronize()
        return
    if args.batched_only:
        from paper_2609_35465_b200 import synth, tetra
        m = shapes.CONFIG4
        one = DevicePass([shapes.Matrix("sweep%d" % i, m.N, m.K) for i in range(12)], seed=args.seed + 13)
        ws = torch.empty(tetra.tetra_batched_workspace_bytes(m.N, m.K), dtype=torch.uint8, device="cuda")
        xb = torch.from_numpy(synth.activations(args.seed + 13, 0, m.K, args.batched_only)).cuda()
        yb = torch.empty((args.batched_only, m.N), dtype=torch.float32, device="cuda")
        for _ in range(2):
            for it in one.items:
                tetra.tetra_gemv_batched(it["codes"], it["row_scales"], one.table, xb, yb, m.N, m.K,
                                         args.batched_only, it["tail"], ws)
        torch.cuda.synchronize()
        return

    model = shapes.MODELS[args.model]
    mats = model.all_matrices()
    if args.layers:
        mats = mats[:7 * args.layers]
    extras = not args.no_extras and rank == 0
    dp = DevicePass(mats, seed=args.seed + 1000 * rank, tail_mode=True, keep_file_codes=extras)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- headline: the whole pass as one persistent grouped launch ---------
    # Rounds of exactly `steps` passes each, CUDA events around every round; as many rounds as it takes to
    # time half a second of work (one round when `steps` alone covers that).  The reported step time is
    # the median round's.
    for _ in range(args.warmup):
        dp.run_grouped()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    round_ms = []
    total_ms = 0.0
    while True:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            dp.run_grouped()
        e1.record(stream)
        barrier()
        t = ranks.max_over_ranks(e0.elapsed_time(e1), device="cuda")
        round_ms.append(t / args.steps)
        total_ms += t
        if total_ms >= 500.0 or len(round_ms) >= 200:
            break
    clocks = sampler.stop()
    ms = float(np.median(round_ms))
    y_grouped = dp.y_all.cpu().numpy().copy()

    # ---- end to end: activations from pinned host memory, results back to it
    e2e_steps = max(3, min(args.steps, 200))
    staged_ms = ranks.max_over_ranks(timed(torch, dp.run_grouped_hostio, e2e_steps, 3, stream), device="cuda")
    y_staged = dp.y_host.numpy().copy()
    dp.plan_mapped_results()
    e2e_ms = ranks.max_over_ranks(timed(torch, dp.run_grouped_mapped, e2e_steps, 3, stream), device="cuda")
    torch.cuda.synchronize()
    assert np.array_equal(dp.y_mapped.numpy(), y_staged), "mapped results differ from the staged copy"
    assert np.array_equal(dp.y_host.numpy(), y_grouped), "host-io result differs from the device-resident run"

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    gbs = dp.algorithmic_bytes / (ms * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": gbs * world, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8 products, int32 block sums, f32 accumulation", "data": "synthetic",
        "config": {"workload": "%s batch-1 weight pass, %d matrices%s" % (
                       model.name, len(mats), "" if not args.layers else " (first %d layers)" % args.layers),
                   "launch": "planned list, two launches per pass (tetra_gemv_grouped_run: activation pre-pass + persistent GEMV)",
                   "k_rule": "floor(K/24) words + float16 tail (the paper's rule)",
                   "l2": "inputs larger than L2: %.2f GB read per pass" % (dp.algorithmic_bytes / 1e9),
                   "seed": args.seed},
        "us_per_pass": ms * 1e3,
        "weights_per_s": sum(m.N * m.K for m in mats) / (ms * 1e-3) * world,
        "bits_per_weight_read": dp.algorithmic_bytes * 8 / sum(m.N * m.K for m in mats),
        "algorithmic_bytes_per_pass": dp.algorithmic_bytes,
        "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS,
        "gpu_launches": 2 * args.steps * len(round_ms),
        "timed_rounds": {"rounds": len(round_ms), "steps_per_round": args.steps, "timed_ms_total": total_ms,
                         "ms_per_step_median": ms, "ms_per_step_best": float(min(round_ms)),
                         "ms_per_step_worst": float(max(round_ms))},
        "clocks": clocks,
        "e2e": {"value": dp.algorithmic_bytes / (e2e_ms * 1e-3) / 1e9 * world, "unit": UNIT,
                "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": int(dp.x_host.numel() * 2),
                "d2h_bytes_per_step": int(dp.y_host.numel() * 4),
                "api": "tetra_gemv_grouped_hostio, mapped results: activations copied from pinned host memory, "
                       "results stored by the kernels into pinned host memory while they run; codes, scales and "
                       "tails stay resident in HBM as model weights do",
                "staged_ms_per_step": staged_ms,
                "staged_note": "same call with a device result buffer and one copy out afterwards"},
        "roofline": {"bound": "hbm", "kernel": "k_gemv_units", "achieved": gbs, "peak": peak, "unit": "GB/s",
                     "frac": gbs / peak, "peak_kind": peak_kind + " copy bandwidth",
                     "traffic": (None if TRAFFIC_PER_ALGORITHMIC_BYTE is None
                                 else TRAFFIC_PER_ALGORITHMIC_BYTE * dp.algorithmic_bytes),
                     "limiter": "instruction issue, not HBM: %.1f warp-instructions per 32 blocks (logic/permute "
                                "pipe %.1f, integer multiply-add pipe %.1f, load/store %.1f; both arithmetic pipes "
                                "take one warp-instruction every two cycles per SM sub-partition); shared-memory "
                                "data pipe %.0f wavefronts per 32 blocks" % (
                                    KERNEL_COUNTERS["instr"], KERNEL_COUNTERS["alu"], KERNEL_COUNTERS["fmaheavy"],
                                    KERNEL_COUNTERS["lsu"], KERNEL_COUNTERS["wavefronts"]),
                     "issue_bound_gbs": issue_bound_gbs(clocks.get("sm_max_mhz") or 1965),
                     "counters_per_32_blocks": KERNEL_COUNTERS},
        "paper_context": {"L40S_tokens_per_s": [113.8, 95.0, 57.2], "L40S_bits_per_weight": 2.148,
                          "L40S_kernel_GBps": 278},
    }

    if extras:
        # secondary arms, a few repetitions each (not part of `value`)
        reps = max(3, min(50, args.steps))
        arms = {}
        arms["per_matrix_stream_ms"] = timed(torch, dp.run_per_matrix, reps, 3, stream)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=torch.cuda.Stream()):
            dp.run_per_matrix(stream=torch.cuda.current_stream())
        arms["per_matrix_graph_ms"] = timed(torch, g.replay, reps, 3, stream)
        y_single = dp.y_all.cpu().numpy()
        assert np.linalg.norm(y_single - y_grouped) <= 1e-5 * np.linalg.norm(y_grouped), \
            "per-matrix launches differ from the planned run"
        arms["paper_design_stream_ms"] = timed(torch, dp.run_paper_design, max(3, reps // 5), 2, stream)
        # the pass as a model would issue it: per layer four dependency steps in stream order (q, k, v | o |
        # gate, up | down: the matrices of a step share their input and are independent, the steps depend on
        # each other), the whole sequence replayed from one CUDA graph.  Each step is one tetra_gemv_list
        # launch; for comparison, the same steps as planned lists (two launches each).
        if not args.layers or args.layers >= 1:
            steps_of_layer = ((0, 3), (3, 4), (4, 6), (6, 7))
            lists = [tetra_mod.make_problems(dp.items[lo + a:lo + b])
                     for lo in range(0, len(dp.items), 7) for a, b in steps_of_layer]

            def run_lists(stream=None):
                for pr in lists:
                    tetra_mod.tetra_gemv_list(pr, dp.table, stream=stream)
            dp.y_all.zero_()
            run_lists()
            torch.cuda.synchronize()
            y_lists = dp.y_all.cpu().numpy()
            assert np.linalg.norm(y_lists - y_grouped) <= 1e-5 * np.linalg.norm(y_grouped), \
                "list launches differ from the planned run"
            gl_ = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gl_, stream=torch.cuda.Stream()):
                run_lists(stream=torch.cuda.current_stream())
            arms["layer_sequence_graph_ms"] = timed(torch, gl_.replay, reps, 3, stream)
            arms["layer_sequence_stream_ms"] = timed(torch, run_lists, reps, 3, stream)
            del gl_
            seq = []
            for pr in lists:
                wsq = torch.empty(max(16, tetra_mod.tetra_grouped_workspace_bytes(pr)), dtype=torch.uint8, device="cuda")
                tetra_mod.tetra_gemv_grouped_plan(pr, wsq)
                seq.append(wsq)
            torch.cuda.synchronize()

            def run_sequence(stream=None):
                for wsq in seq:
                    tetra_mod.tetra_gemv_grouped_run(wsq, dp.table, stream=stream)
            run_sequence()
            gs_ = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gs_, stream=torch.cuda.Stream()):
                run_sequence(stream=torch.cuda.current_stream())
            arms["layer_sequence_planned_lists_graph_ms"] = timed(torch, gs_.replay, reps, 3, stream)
            out["layer_sequence"] = {"steps_per_pass": len(lists), "launches_per_pass": len(lists),
                                     "note": "four dependent steps per layer (q,k,v | o | gate,up | down), one "
                                             "tetra_gemv_list launch each; planned lists take two launches each"}
            del gs_, seq
            dp.run_grouped()
            torch.cuda.synchronize()
        # 20 rounds of ten planned passes each: median and best round (the paper reports the median of its rounds)
        rounds = sorted(timed(torch, dp.run_grouped, 10, 0, stream) for _ in range(20))
        out["rounds_of_10_steps"] = {"median_ms": rounds[len(rounds) // 2], "best_ms": rounds[0], "worst_ms": rounds[-1]}
        # launch-overhead control (Sec. 5.2's "no weights" arm): the same 252 single-matrix launches on
        # matrices cut down to one block and a 16-weight tail per row (K = 40), i.e. next to no code reads
        ctl = DevicePass([shapes.Matrix(m.name, m.N, 40) for m in mats], seed=args.seed + 19)
        arms["no_weights_control_stream_ms"] = timed(torch, ctl.run_per_matrix, reps, 3, stream)
        gc = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gc, stream=torch.cuda.Stream()):
            ctl.run_per_matrix(stream=torch.cuda.current_stream())
        arms["no_weights_control_graph_ms"] = timed(torch, gc.replay, reps, 3, stream)
        del gc, ctl
        for k in list(arms):
            if not k.startswith("no_weights"):
                arms[k.replace("_ms", "_GBps")] = dp.algorithmic_bytes / (arms[k] * 1e-3) / 1e9
        out["other_arms"] = arms
        for k in ("layer_sequence_graph_ms", "per_matrix_graph_ms", "no_weights_control_graph_ms"):
            if k in arms:
                out[k] = arms[k]       # beside `value`: the pass in model order, and one launch per matrix
        dp.run_grouped()
        torch.cuda.synchronize()

        # microseconds per matrix of the single-matrix entry point (tetra_gemv_tail), per shape of a layer:
        # distinct copies of the shape, together more than twice the 126 MB L2, replayed from a CUDA graph, so
        # no launch reads L2-resident codes
        peak_now = measured_peak()[0]
        L2_BYTES = 126e6

        def copies_for(nbytes):
            return int(max(12, min(400, np.ceil(2.2 * L2_BYTES / nbytes))))

        def time_shape(mats_of_copy, run_name):
            """mats_of_copy: shapes of one copy; returns (microseconds per copy, bytes per copy, copies)."""
            probe = sum(m.N * (m.blocks * 6 + m.ntail * 2 + 8) + m.K * 2 for m in mats_of_copy)
            copies = copies_for(probe)
            one = DevicePass([shapes.Matrix("%s_%d" % (m.name, i), m.N, m.K) for i in range(copies) for m in mats_of_copy],
                             seed=args.seed + 7)
            n = len(mats_of_copy)
            if run_name == "per_matrix":
                fn = one.run_per_matrix
            else:
                groups = [tetra_mod.make_problems(one.items[i * n:(i + 1) * n]) for i in range(copies)]

                def fn(stream=None):
                    for pr in groups:
                        tetra_mod.tetra_gemv_list(pr, one.table, stream=stream)
            for _ in range(2):
                fn()
            gg = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gg, stream=torch.cuda.Stream()):
                fn(stream=torch.cuda.current_stream())
            us = timed(torch, gg.replay, 20, 3, stream) * 1e3 / copies
            b = sum(it["bytes"] for it in one.items[:n])
            del one, gg
            torch.cuda.empty_cache()
            return us, b, copies

        def figure(mats_of_copy, run_name):
            us, b, copies = time_shape(mats_of_copy, run_name)
            return {"us": us, "GBps": b / us / 1e3, "algorithmic_bytes": b, "distinct_copies": copies,
                    "weights_per_s": sum(m.N * m.K for m in mats_of_copy) / us * 1e6,
                    "frac_of_measured_peak": b / us / 1e3 / peak_now, "roofline_us": b / peak_now / 1e3}

        per_matrix = {}
        for m in model.layer_matrices():
            per_matrix[m.name] = dict(figure([m], "per_matrix"), N=m.N, K=m.K)
        out["per_matrix_tetra_gemv"] = per_matrix
        # BASELINE configs 0 and 1: the single 2048 x 2304 matrix (one launch), and one Qwen3-4B-shaped layer
        # (seven matrices) as its four dependency steps, one tetra_gemv_list launch each
        l4 = shapes.QWEN3_4B.layer_matrices()
        cfg1 = {"us_per_layer": 0.0, "algorithmic_bytes": 0, "launches": 4}
        for a, b in ((0, 3), (3, 4), (4, 6), (6, 7)):
            f = figure(l4[a:b], "list")
            cfg1["us_per_layer"] += f["us"]
            cfg1["algorithmic_bytes"] += f["algorithmic_bytes"]
            cfg1["+".join(m.name for m in l4[a:b])] = {"us": f["us"], "GBps": f["GBps"]}
        cfg1["GBps"] = cfg1["algorithmic_bytes"] / cfg1["us_per_layer"] / 1e3
        cfg1["frac_of_measured_peak"] = cfg1["GBps"] / peak_now
        out["configs"] = {"config0_2048x2304": dict(figure([shapes.CONFIG0], "per_matrix"), N=shapes.CONFIG0.N, K=shapes.CONFIG0.K),
                          "config1_qwen3_4b_layer": cfg1}

        # batch sweep on the down_proj shape (N 4096, K 12288): tetra_gemv_batched (decode once, tensor-core
        # contraction) against one tetra_gemv_tail launch per vector; 12 distinct code copies per CUDA graph
        from paper_2609_35465_b200 import synth, tetra
        m = shapes.CONFIG4
        sweep = {}
        one = DevicePass([shapes.Matrix("sweep%d" % i, m.N, m.K) for i in range(12)], seed=args.seed + 13)
        ws = torch.empty(tetra.tetra_batched_workspace_bytes(m.N, m.K), dtype=torch.uint8, device="cuda")
        for batch in shapes.CONFIG4_BATCHES:
            xb = torch.from_numpy(synth.activations(args.seed + 13, 0, m.K, batch)).cuda()
            yb = torch.empty((batch, m.N), dtype=torch.float32, device="cuda")

            def run_batched(stream=None):
                for it in one.items:
                    tetra.tetra_gemv_batched(it["codes"], it["row_scales"], one.table, xb, yb, m.N, m.K, batch,
                                             it["tail"], ws, stream=stream)

            def run_loop(stream=None):
                for it in one.items:
                    for v in range(batch):
                        tetra.tetra_gemv_tail(it["codes"], it["row_scales"], one.table, xb[v], yb[v], m.N, m.K, 1,
                                              it["tail"], stream=stream)
            us = {}
            for name, fn in (("batched", run_batched), ("per_vector", run_loop)):
                fn()
                gg = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gg, stream=torch.cuda.Stream()):
                    fn(stream=torch.cuda.current_stream())
                us[name] = timed(torch, gg.replay, 10, 3, stream) * 1e3 / 12
                del gg
            sweep[str(batch)] = {"batched_us": us["batched"], "per_vector_launches_us": us["per_vector"],
                                 "us_per_vector": us["batched"] / batch,
                                 "weights_x_vectors_per_s": m.N * m.K * batch / us["batched"] * 1e6}
        t1 = sweep["1"]
        sweep["first_batch_over_1p25x_batch1_time"] = {
            "batched": next((b for b in shapes.CONFIG4_BATCHES if sweep[str(b)]["batched_us"] > 1.25 * t1["batched_us"]), None),
            "per_vector_launches": next((b for b in shapes.CONFIG4_BATCHES
                                         if sweep[str(b)]["per_vector_launches_us"] > 1.25 * t1["per_vector_launches_us"]), None)}
        out["batch_sweep_4096x12288"] = sweep
        del one, ws

        # 4-bit group-quantised matrices (the served model's other weight format): the int4 projection shapes
        # of this model (groups of 128) and the output head (151,936 rows, groups of 64), batch 1, CUDA graph
        # over distinct copies (more than L2 together), after half a second of the same work
        q4 = {}
        kv_dim, q_dim = model.kv_heads * model.head_dim, model.q_heads * model.head_dim
        q4_shapes = [("v_proj", kv_dim, model.hidden, 128, 48), ("o_proj", model.hidden, q_dim, 128, 24),
                     ("down_proj", model.hidden, model.intermediate, 128, 12),
                     ("head", 151936, model.hidden, 64, 2)]
        for name, qN, qK, qG, copies in q4_shapes:
            rows_src = min(qN, 4096)  # the head repeats a 4096-row pattern of nibbles: timing only
            qn = torch.from_numpy(synth.q4_nibbles(args.seed + 17, qN, rows_src, qK)).cuda()
            qn = qn.repeat((qN + rows_src - 1) // rows_src, 1)[:qN].contiguous()
            sc, of = synth.q4_scales_offsets(args.seed + 17, qN, qN, qK // qG)
            sc, of = torch.from_numpy(sc).cuda(), torch.from_numpy(of).cuda()
            packs = [tetra.tetra_q4_pack(qn, sc, of, qN, qK, qG) for _ in range(copies)]
            xq = torch.from_numpy(synth.activations(args.seed + 17, 1, qK, 1)).cuda()
            yq = torch.empty((1, qN), dtype=torch.float32, device="cuda")

            def run_q4(stream=None):
                for pk in packs:
                    tetra.tetra_q4_gemv(pk, xq, yq, qN, qK, qG, 1, stream=stream)
            run_q4()
            gg = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gg, stream=torch.cuda.Stream()):
                run_q4(stream=torch.cuda.current_stream())
            us_burst = timed(torch, gg.replay, 20, 3, stream) * 1e3 / copies  # from idle, as the copy peak was measured
            t_end = time.time() + 0.5
            while time.time() < t_end:
                gg.replay()
                torch.cuda.synchronize()
            us = timed(torch, gg.replay, 20, 3, stream) * 1e3 / copies        # sustained (power limit, lower SM clock)
            nbytes = packs[0].numel() + 2 * qK + 4 * qN
            q4[name] = {"N": qN, "K": qK, "group": qG, "us": us, "algorithmic_bytes": nbytes, "GBps": nbytes / us / 1e3,
                        "frac_of_measured_peak": nbytes / us / 1e3 / peak_now, "roofline_us": nbytes / peak_now / 1e3,
                        "us_burst": us_burst, "GBps_burst": nbytes / us_burst / 1e3,
                        "frac_of_measured_peak_burst": nbytes / us_burst / 1e3 / peak_now,
                        "bits_per_weight": 8.0 * packs[0].numel() / (qN * qK)}
            del packs, gg, qn, sc, of
            torch.cuda.empty_cache()
        # the same projection shapes as ONE planned list (v, o and down of every layer: 3 x layers matrices,
        # distinct copies, more than L2 together), three launches per pass (tetra_q4_list_run)
        qitems = []
        for layer in range(model.layers):
            for name, qN, qK, qG, _ in q4_shapes[:3]:
                rows_src = min(qN, 4096)
                qn = torch.from_numpy(synth.q4_nibbles(args.seed + 17, qN, rows_src, qK)).cuda()
                sc, of = synth.q4_scales_offsets(args.seed + 17, qN, qN, qK // qG)
                pk = tetra.tetra_q4_pack(qn, torch.from_numpy(sc).cuda(), torch.from_numpy(of).cuda(), qN, qK, qG)
                qitems.append(dict(packed=pk, N=qN, K=qK,
                                   x=torch.from_numpy(synth.activations(args.seed + 17, layer, qK, 1)[0]).cuda(),
                                   y=torch.empty(qN, dtype=torch.float32, device="cuda")))
                del qn
        qprob = tetra.make_q4_problems(qitems)
        qws = tetra.tetra_q4_list_plan(qprob, 128)
        torch.cuda.synchronize()
        # a burst of 20 passes first (as the copy-bandwidth peak was measured), then the same after half a
        # second of this work: at 5 TB/s with the tensor cores busy the board reaches its power limit and the
        # SM clock drops, so the sustained figure is the lower one
        ms_list_burst = timed(torch, lambda: tetra.tetra_q4_list_run(qws, 128), 20, 3, stream)
        t_end = time.time() + 0.5
        while time.time() < t_end:
            tetra.tetra_q4_list_run(qws, 128)
            torch.cuda.synchronize()
        ms_list = timed(torch, lambda: tetra.tetra_q4_list_run(qws, 128), 20, 3, stream)
        # spot check against the single-matrix entry point (itself checked against the oracle in the tests)
        it0 = qitems[5]
        y1 = torch.empty((1, it0["N"]), dtype=torch.float32, device="cuda")
        tetra.tetra_q4_gemv(it0["packed"], it0["x"].reshape(1, -1), y1, it0["N"], it0["K"], 128, 1)
        torch.cuda.synchronize()
        assert torch.linalg.norm(y1[0] - it0["y"]) <= 1e-5 * torch.linalg.norm(y1[0]), "q4 list differs from q4 gemv"
        nbytes_list = sum(it["packed"].numel() + 2 * it["K"] + 4 * it["N"] for it in qitems)
        q4["planned_list_v_o_down"] = {"matrices": len(qitems), "algorithmic_bytes": nbytes_list, "ms_per_pass": ms_list,
                                       "GBps": nbytes_list / (ms_list * 1e-3) / 1e9,
                                       "frac_of_measured_peak": nbytes_list / (ms_list * 1e-3) / 1e9 / peak_now,
                                       "ms_per_pass_burst": ms_list_burst,
                                       "GBps_burst": nbytes_list / (ms_list_burst * 1e-3) / 1e9,
                                       "frac_of_measured_peak_burst": nbytes_list / (ms_list_burst * 1e-3) / 1e9 / peak_now,
                                       "note": "ms_per_pass after half a second of the same work (power limit reached, SM clock "
                                               "below its maximum); the burst figure is 20 passes from idle",
                                       "single_launches_sum_ms": sum(q4[n]["us"] for n in ("v_proj", "o_proj", "down_proj"))
                                                                 * model.layers * 1e-3,
                                       "launches_per_pass": 3}
        del qitems, qws
        torch.cuda.empty_cache()
        out["q4_gemv"] = q4

        # encoder search on Gaussian blocks (Sec. 3.5): exact largest-cosine point per block on the GPU, and the
        # oracle's exact search on a bounded sample of the same blocks on the host cores
        from oracle import encode as oenc
        n_enc = 20000
        w_enc = synth.normal(11, 0, 20, n_enc * 24).reshape(n_enc, 24).astype(np.float32)
        wd = torch.from_numpy(w_enc).cuda()
        enc_table = tetra.tetra_build_table(synth.DEFAULT_GAIN)
        tetra.tetra_encode_blocks(wd, enc_table)
        t_enc = timed(torch, lambda: tetra.tetra_encode_blocks(wd, enc_table), 3, 1, stream)
        codes_enc, cos_enc = tetra.tetra_encode_blocks(wd, enc_table)
        torch.cuda.synchronize()
        t0 = time.time()
        _, cos_ref = oenc.encode_blocks(w_enc[:256].astype(np.float64))
        t_ref = time.time() - t0
        out["encoder"] = {"blocks": n_enc, "ms": t_enc, "blocks_per_s": n_enc / (t_enc * 1e-3),
                          "mean_cosine": float(cos_enc.mean().item()),
                          "oracle_blocks_per_s": 256 / t_ref, "oracle_cores": os.cpu_count() or 1,
                          "max_abs_cosine_difference_on_oracle_sample":
                              float(np.max(np.abs(cos_enc[:256].cpu().numpy().astype(np.float64) - cos_ref)))}

        # the other two model sizes, planned-list pass (same kernels; a few repetitions)
        others = {}
        for name in ("qwen3-4b", "qwen3-14b"):
            if name == model.name or args.layers:
                continue
            mm = shapes.MODELS[name]
            od = DevicePass(mm.all_matrices(), seed=args.seed + 11)
            # correctness first (Sec. 5.1): sampled rows of every matrix of the pass against the oracle
            od.run_grouped()
            torch.cuda.synchronize()
            y_od = od.y_all.cpu().numpy()
            import oracle
            from oracle.check import gemv_errors, oracle_product
            worst_od = 0.0
            for i, it in enumerate(od.items):
                rows = np.unique(np.concatenate([[0, it["N"] - 1],
                                                 np.random.default_rng(args.seed + i).integers(0, it["N"], 6)]))
                ref = oracle_product(oracle.get(), od.host_inputs(i, rows), od.gain)
                rel, worst = gemv_errors(y_od[it["yoff"] + rows], ref)
                worst_od = max(worst_od, worst, rel / 1e-3)
            if worst_od > 1.0:
                raise SystemExit("%s pass outside the tolerance on sampled rows: %.3f" % (name, worst_od))
            t = timed(torch, od.run_grouped, 30, 3, stream)
            others[name] = {"matrices": len(od.items), "algorithmic_bytes": od.algorithmic_bytes, "ms_per_pass": t,
                            "sampled_rows_worst_fraction_of_tolerance": worst_od,
                            "GBps": od.algorithmic_bytes / (t * 1e-3) / 1e9,
                            "frac_of_measured_peak": od.algorithmic_bytes / (t * 1e-3) / 1e9 / peak_now,
                            "weights_per_s": sum(x.N * x.K for x in mm.all_matrices()) / (t * 1e-3)}
            del od
            torch.cuda.empty_cache()
        out["other_models"] = others

        # CPU baseline: the oracle on a bounded sample of the same pass, all host cores
        import oracle
        orc = oracle.get()
        cores = os.cpu_count() or 1
        dt1, b1, _, _ = oracle_sample(dp, orc, 1, cores)
        layers = int(max(1, min(model.layers if not args.layers else args.layers, 12.0 / max(dt1, 1e-3))))
        dt, nb, worst, nmat = oracle_sample(dp, orc, layers, cores, compare_with=y_grouped)
        out["cpu_baseline"] = {"value": nb / dt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
                               "sample": "first %d layers (%d matrices, %.3f GB) of the same pass, %.1f s"
                                         % (layers, nmat, nb / 1e9, dt),
                               "gpu_vs_oracle_worst_fraction_of_tolerance": worst}
        if worst is not None and worst > 1.0:
            raise SystemExit("GPU result outside the tolerance on the CPU-baseline sample: %.3f" % worst)
        dts, nbs, _, nms = oracle_sample(dp, orc, 1, 1)
        out["cpu_baseline_single_thread"] = {"value": nbs / dts / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
                                             "sample": "first layer (%d matrices, %.3f GB), %.1f s" % (nms, nbs / 1e9, dts)}

    print(json.dumps(out))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
