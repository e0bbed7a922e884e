#!/usr/bin/env python
"""Benchmark of the per-epoch KV-cache management pass.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one epoch of the whole hot path on one pool: event reduction + EMA +
posterior + score and k-lowest selection (kv_epoch_score_select: two launches),
pack + D2H to the pinned host ring (kv_demote), H2D + unpack of prefetched
entries (kv_promote).  Admission of fresh blocks, which keeps the pool full, is
a harness step and runs untimed between steps, as does an L2 flush.

By default the pool is the largest of the five that fits the device and the
pinned host tier (the mixed fleet of 150 GiB, else the 90 GiB long-context pool,
scaled down by a recorded factor only when free memory says so); --config picks
one by number.

Prints ONE JSON line.  `value` is KV head-blocks scored + selected per second,
N / t(scoring + selection), measured inside full steps; `roofline` is that
pass against the HBM peak; the line also carries the whole-step rate, per-phase
bandwidths (pack / unpack kernels against HBM, copies against the host link
measured in the same run), and the CPU oracle timed on the host cores.
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

METRIC = "KV head-blocks scored+selected/s"
UNIT = "head-blocks/s"

# DRAM traffic from ncu (dram__bytes_read.sum + dram__bytes_write.sum) per payload
# byte of a pack launch: captured on a 256 MiB payload-only
# launch of a 3 GiB pool (487.35 MB of traffic for 268.44 MB of payload) and
# scaled to the benchmark's launch size in proportion to the payload.
NCU_PACK_TRAFFIC_BYTES_PER_PAYLOAD_BYTE = 487.35 / 268.44
PACK_KERNEL_NAME = "move_tma_kernel<true> (pack)"

# DRAM traffic of the scoring + selection pass (event_reduce_kernel followed by
# select_persistent_kernel<true>) from ncu, bytes per launch pair, keyed by pool number: captured
# at the pool's full entry count with --tiny-entries (these kernels never touch block payload).
# None = no capture of the kernels as they stand.  (ncu flushes the caches before every kernel it
# replays: the figures are those of a cold L2, without what kv_set_l2_residency keeps there.)
NCU_SCORE_SELECT_TRAFFIC = {5: 547.2e6, 3: 438.7e6}


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=None,
                    help="pool 1..5 (default: the largest that fits device memory and the pinned host tier)")
    ap.add_argument("--scale", type=float, default=None,
                    help="shrinks blocks per layer (default: 1, or what free memory allows)")
    ap.add_argument("--ring-slots", type=int, default=None)
    ap.add_argument("--batch-mb", type=int, default=1320,
                    help="demote/promote chunk (staging buffer) size; the default lets the default pool's demotion "
                         "(2.58 GB) take two chunks, so that both pack launches run back to back")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-hostlink", action="store_true", help="skip the 1 GiB host-link probe")
    ap.add_argument("--no-deferred-packing", action="store_true",
                    help="enqueue the whole demotion before the promotion instead of interleaving their chunks")
    ap.add_argument("--sharded", action="store_true",
                    help="use the sharded epoch path (kv_epoch_events + all-reduce + kv_epoch_update) even on one rank")
    ap.add_argument("--no-fused", action="store_true",
                    help="score and select with two calls (kv_epoch_score, kv_select_victims) instead of the fused one")
    ap.add_argument("--head-weights", action="store_true",
                    help="update every partition's head-importance matrix each step and weight the scores with it")
    ap.add_argument("--no-breakdown", action="store_true",
                    help="skip the three extra epochs that time event reduction, entry pass and selection one by one")
    ap.add_argument("--dedup", action="store_true",
                    help="after the timed steps, also time content hashing (SHA-256 of every entry) and "
                         "deduplication of the digests; reported under phases, not part of a step")
    ap.add_argument("--tiny-entries", action="store_true",
                    help="32-64 byte blocks (same entry count and traces): for profiling scoring/selection")
    ap.add_argument("--promote-run", type=int, default=None,
                    help="promote lists made of runs of exactly this many consecutive ring slots at seeded places "
                         "(instead of the pool's own list style)")
    ap.add_argument("--gather-kb", type=int, default=None,
                    help="promote lists whose runs average less than this many KiB go through the gather kernel "
                         "(0 = always one transfer per run; default: the library's 256)")
    ap.add_argument("--l2-mb", type=int, default=48,
                    help="budget of kv_set_l2_residency in MiB: one state array (touch counts, else pair bytes) kept "
                         "in the persisting part of the L2 for the scoring kernels; 0 = off")
    ap.add_argument("--select-variant", type=int, default=1, choices=[0, 1],
                    help="selection: 1 = one persistent cooperative launch, 0 = one launch per phase")
    return ap.parse_args()


def device_need_bytes(w, batch_bytes):
    """Device memory a pool of this workload takes in the benchmark (slabs, four staging
    buffers, per-entry state and workspace, block table, the L2-flush buffer, victims)."""
    per_entry = 26 + 4 + 8 + 4      # state arrays, free list, tile scratch, victim list
    return (sum(p.slab_bytes for p in w.parts) + 4 * (batch_bytes + (batch_bytes // 8192 + 2) * 24 + 64)
            + w.N * per_entry + w.n_tags * 4 + sum(p.ring_slots for p in w.parts) * 21 + (256 << 20) + (1 << 30))


def host_need_bytes(w):
    return sum(p.ring_slots * (p.entry_bytes + 24) for p in w.parts) + (2 << 30)


def choose_workload(args, torch, W, dev):
    """The workload to run: --config / --scale if given, else the largest pool that fits."""
    def make(cfg, scale):
        return W.config(cfg, scale=scale, ring_slots=args.ring_slots, tiny_entries=args.tiny_entries)
    if args.config is not None:
        scale = 1.0 if args.scale is None else args.scale
        return args.config, scale, make(args.config, scale), "--config"
    free_dev, _ = torch.cuda.mem_get_info(dev)
    try:
        import psutil
        free_host = psutil.virtual_memory().available
    except Exception:
        free_host = os.sysconf("SC_PAGE_SIZE") * os.sysconf("SC_AVPHYS_PAGES")
    batch = args.batch_mb << 20
    why = ""
    for cfg in (5, 3, 2):
        scale = 1.0 if args.scale is None else args.scale
        w = make(cfg, scale)
        fit = min(1.0, 0.97 * free_dev / device_need_bytes(w, batch), 0.6 * free_host / host_need_bytes(w))
        if fit >= 1.0:
            return cfg, scale, w, why + "pool %d fits: %.0f GiB free on the device, %.0f GiB free on the host" % (
                cfg, free_dev / 2**30, free_host / 2**30)
        if args.scale is None and fit >= 0.5:
            scale = int(fit * 20) / 20.0      # in steps of 0.05, rounded down
            return cfg, scale, make(cfg, scale), why + (
                "pool %d scaled by %.2f: %.0f GiB free on the device, %.0f GiB free on the host" % (
                    cfg, scale, free_dev / 2**30, free_host / 2**30))
        why += "pool %d does not fit (needs %.0f GiB device, %.0f GiB pinned host); " % (
            cfg, device_need_bytes(w, batch) / 2**30, host_need_bytes(w) / 2**30)
    return 2, 1.0, make(2, 1.0), why


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while running."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.lines = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "200"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        for ln in self.lines:
            c = [x.strip() for x in ln.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1]))
                smax.append(float(c[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                  "sw_power_cap"), c[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def hostlink_probe(torch, dev, nbytes=1 << 30, reps=10):
    """cudaMemcpyAsync of 1 GiB pinned<->device, best of `reps`, CUDA events."""
    h = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    d = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    h2 = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    d2 = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    s1, s2 = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    out = {}

    def run(fn, streams):
        best = 1e30
        for _ in range(reps):
            torch.cuda.synchronize(dev)
            a = [torch.cuda.Event(enable_timing=True) for _ in streams]
            b = [torch.cuda.Event(enable_timing=True) for _ in streams]
            for i, s in enumerate(streams):
                a[i].record(s)
            fn()
            for i, s in enumerate(streams):
                b[i].record(s)
            torch.cuda.synchronize(dev)
            best = min(best, max(x.elapsed_time(y) for x, y in zip(a, b)))
        return best

    def d2h():
        with torch.cuda.stream(s1):
            h.copy_(d, non_blocking=True)

    def h2d():
        with torch.cuda.stream(s1):
            d.copy_(h, non_blocking=True)

    def both():
        with torch.cuda.stream(s1):
            h.copy_(d, non_blocking=True)
        with torch.cuda.stream(s2):
            d2.copy_(h2, non_blocking=True)

    out["d2h_gbs"] = nbytes / run(d2h, [s1]) / 1e6
    out["h2d_gbs"] = nbytes / run(h2d, [s1]) / 1e6
    out["bidir_gbs_per_dir"] = nbytes / run(both, [s1, s2]) / 1e6
    out["how"] = "1 GiB pinned<->device copies, best of %d, CUDA events" % reps
    del h, d, h2, d2
    return out


# Integer-pipe slots of one SHA-256 compression (64 bytes) as the kernel issues it: 64 rounds of
# 6 funnel shifts + 4 three-input logic ops, 48 schedule steps of 6 shifts + 2 logic ops, 16 byte
# swaps; a funnel shift issues at half the rate of the others, so it takes two slots.  The
# additions are issued as multiply-adds on the FMA pipe and do not queue here.  An SM issues 128
# lanes per clock (4 schedulers x 32).
SHA_SLOTS_PER_64B = 64 * (2 * 6 + 4) + 48 * (2 * 6 + 2) + 16


def time_dedup(torch, pool, w, B, reps=3):
    """Times kv_hash_entries over every entry and kv_dedup_digests over the digests."""
    N = w.N
    dev = pool.device
    d = torch.zeros((N, 32), dtype=torch.uint8, device=dev)
    table = torch.empty(B.kv_dedup_table_slots(N), dtype=torch.int32, device=dev)
    canon = torch.empty(N, dtype=torch.int32, device=dev)
    ref = torch.empty(N, dtype=torch.int32, device=dev)
    extra = torch.zeros(8, dtype=torch.int32, device=dev)
    t_hash, t_dedup = [], []
    for _ in range(reps):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        ev[0].record(pool.compute)
        rc = pool.kv_hash_entries(None, N, d)
        ev[1].record(pool.compute)
        rc2 = B.kv_dedup_digests(d, N, canon, ref, table, extra[0:], extra[4:], pool.compute)
        ev[2].record(pool.compute)
        torch.cuda.synchronize(dev)
        if rc != B.KV_OK or rc2 != B.KV_OK:
            raise B.KVError(rc or rc2, "kv_hash_entries / kv_dedup_digests")
        t_hash.append(ev[0].elapsed_time(ev[1]))
        t_dedup.append(ev[1].elapsed_time(ev[2]))
    nbytes = sum(p.slab_bytes for p in w.parts)
    gbs = nbytes / min(t_hash) / 1e6
    sm_clock_ghz = 1.965     # clocks.max.sm; the kernel draws far less than the power cap
    alu_peak_gbs = 148 * 128 * sm_clock_ghz * 64 / SHA_SLOTS_PER_64B
    return {"hash_ms": min(t_hash), "hash_gbs": gbs, "hash_alu_peak_gbs": alu_peak_gbs,
            "hash_frac_of_alu_peak": gbs / alu_peak_gbs, "dedup_ms": min(t_dedup),
            "dedup_unique": int(extra[0].item()), "dedup_status": int(extra[4].item())}


def oracle_pool(w):
    from oracle import kv_oracle as O
    parts = [dict(model=O.Model(p.variant, p.n_layers, p.n_q_heads, p.n_kv_heads, p.head_dim,
                                p.d_latent, p.d_rope, p.dtype_bits),
                  block_tokens=p.block_tokens, blocks_per_layer=p.blocks_per_layer,
                  ring_slots=p.ring_slots) for p in w.parts]
    return O, O.OraclePool(parts, w.alpha0, w.beta0, n_tags=w.n_tags, payload=False)


def oracle_epochs(w, n_epochs, warm=0):
    """Times the CPU oracle (metadata mode: state, tables and counters, no payload
    bytes) on the workload.  Returns (seconds in score+select, seconds per full
    epoch, epochs timed)."""
    from paper_2604_26968_b200.harness import INITIAL_EPOCH_KEY
    O, pool = oracle_pool(w)
    fresh = np.flatnonzero(pool.state == O.FREE).astype(np.uint32)
    pool.admit(0, w.decay, w.new_pairs(INITIAL_EPOCH_KEY, fresh.size), None)
    t_ss, t_all, done = 0.0, 0.0, 0
    for e in range(warm + n_epochs):
        ev_entry, ev_hit = w.events(e, pool.pair, fresh)
        t0 = time.perf_counter()
        assert pool.epoch_score(e, ev_entry, ev_hit) == O.OK
        rc, v = pool.select_victims(w.k)
        t1 = time.perf_counter()
        assert rc == O.OK and pool.demote(v) == O.OK
        t_move = time.perf_counter() - t1
        for q, p in enumerate(w.parts):
            inf = pool.info(q)
            live = pool.part_array(q, "r_live")
            n_fq = int((pool.state[inf["base"]:inf["base"] + inf["n"]] == O.FREE).sum())
            m_q = min(int(w.promote_frac * p.n_entries), n_fq, int(live.sum()))
            lst = w.promote_list(e, q, m_q, inf["cursor"], live, just_written=n_fq)
            t2 = time.perf_counter()
            assert pool.promote(q, lst) == O.OK
            t_move += time.perf_counter() - t2
        if e >= warm:
            t_ss += t1 - t0
            t_all += (t1 - t0) + t_move
            done += 1
        fresh = np.flatnonzero(pool.state == O.FREE).astype(np.uint32)
        pool.admit(e, w.decay, w.new_pairs(e, fresh.size), None)
    pool.close()
    return t_ss, t_all, done


def oracle_movement(W, cfg, target_bytes=1 << 30, epochs=3):
    """GB/s of the oracle's memcpy-based demotion and promotion (payload mode, 1 thread)
    on the workload scaled down to about target_bytes of slab."""
    from paper_2604_26968_b200.harness import INITIAL_EPOCH_KEY
    full = W.config(cfg)
    scale = min(1.0, target_bytes / sum(p.slab_bytes for p in full.parts))
    w = W.config(cfg, scale=scale)
    O, _ = None, None
    from oracle import kv_oracle as O
    parts = [dict(model=O.Model(p.variant, p.n_layers, p.n_q_heads, p.n_kv_heads, p.head_dim,
                                p.d_latent, p.d_rope, p.dtype_bits),
                  block_tokens=p.block_tokens, blocks_per_layer=p.blocks_per_layer,
                  ring_slots=p.ring_slots) for p in w.parts]
    pool = O.OraclePool(parts, w.alpha0, w.beta0, n_tags=w.n_tags, payload=True)

    def admit(e, key):
        fresh = np.flatnonzero(pool.state == O.FREE).astype(np.uint32)
        nbytes = 0
        for q in range(pool.n_parts):
            inf = pool.info(q)
            nbytes += int((pool.state[inf["base"]:inf["base"] + inf["n"]] == O.FREE).sum()) * inf["entry_bytes"]
        pool.admit(e, w.decay, w.new_pairs(key, fresh.size), np.zeros(nbytes, np.uint8))
        return fresh

    fresh = admit(0, INITIAL_EPOCH_KEY)
    t_dem = t_pro = 0.0
    b_dem = b_pro = 0
    for e in range(epochs):
        ev_entry, ev_hit = w.events(e, pool.pair, fresh)
        assert pool.epoch_score(e, ev_entry, ev_hit) == O.OK
        rc, v = pool.select_victims(w.k)
        assert rc == O.OK
        s0 = pool.stats()
        t0 = time.perf_counter()
        assert pool.demote(v) == O.OK
        t_dem += time.perf_counter() - t0
        for q, p in enumerate(w.parts):
            inf = pool.info(q)
            live = pool.part_array(q, "r_live")
            n_fq = int((pool.state[inf["base"]:inf["base"] + inf["n"]] == O.FREE).sum())
            m_q = min(int(w.promote_frac * p.n_entries), n_fq, int(live.sum()))
            lst = w.promote_list(e, q, m_q, inf["cursor"], live, just_written=n_fq)
            t0 = time.perf_counter()
            assert pool.promote(q, lst) == O.OK
            t_pro += time.perf_counter() - t0
        s1 = pool.stats()
        b_dem += s1["bytes_demoted"] - s0["bytes_demoted"]
        b_pro += s1["bytes_promoted"] - s0["bytes_promoted"]
        fresh = admit(e, e)
    pool.close()
    return {"demote_gbs": b_dem / max(t_dem, 1e-12) / 1e9, "promote_gbs": b_pro / max(t_pro, 1e-12) / 1e9,
            "pool_bytes": sum(p.slab_bytes for p in w.parts), "scale": scale, "epochs": epochs}


def reference_workload(args, W):
    """The pool the CUDA arm would choose on this machine (asks the device for its free
    memory when one is there; no kernel is launched)."""
    try:
        import torch
        if torch.cuda.is_available():
            local = int(os.environ.get("LOCAL_RANK", "0"))
            return choose_workload(args, torch, W, torch.device("cuda", local))
    except Exception:
        pass
    cfg = args.config if args.config is not None else 5
    scale = args.scale if args.scale is not None else 1.0
    return cfg, scale, W.config(cfg, scale=scale, ring_slots=args.ring_slots, tiny_entries=args.tiny_entries), \
        "no CUDA device to ask"


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2604_26968_b200 import workloads as W
    cfg, scale, w, why = reference_workload(args, W)
    t_ss, t_all, done = oracle_epochs(w, args.steps, warm=args.warmup)
    value = w.N * done / t_ss
    sample = "%d full epochs of pool %d (N=%d) in metadata mode (no payload bytes), 1 thread" % (
        done, cfg, w.N)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_ss / done,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": {"workload": w.name, "pool": cfg, "n_entries": w.N,
                                        "k": w.k, "scale": scale, "chosen_because": why},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": w.N * done / t_all, "unit": UNIT, "scope": "whole epoch (score, select, demote, "
                "promote) in metadata mode: no payload bytes move", "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
        return
    import torch
    import torch.distributed as dist
    from paper_2604_26968_b200 import workloads as W
    from paper_2604_26968_b200.harness import EpochRunner

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist_on = world > 1 or args.sharded    # --sharded: take the multi-GPU code path even on one rank
    if dist_on:
        if "RANK" not in os.environ:      # --sharded started without a launcher: a group of one
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29533")
            os.environ["RANK"], os.environ["WORLD_SIZE"] = "0", "1"
        dist.init_process_group("nccl", device_id=dev)

    cfg, scale, w, chosen_because = choose_workload(args, torch, W, dev)
    w.seed = w.seed + 1000 * rank     # every rank owns its own pool and trace (weak scaling)
    if args.promote_run is not None:
        w.promote_style, w.max_run = "aligned-runs", args.promote_run
    w.epochs = args.warmup + args.steps + 12   # block handles for every epoch this run admits (timed, e2e, breakdown)
    link = hostlink_probe(torch, dev) if rank == 0 and not args.no_hostlink else None
    runner = EpochRunner(w, batch_bytes=args.batch_mb << 20, fill_pattern=True, host_meta=True,
                         device=str(dev))
    pool = runner.pool
    pool.kv_timing_enable(True)
    from paper_2604_26968_b200 import binding as B
    pool.kv_set_select_variant(args.select_variant)
    pool.kv_set_deferred_packing(not args.no_deferred_packing)
    if args.gather_kb is not None:
        pool.kv_set_gather_threshold(args.gather_kb << 10)
    l2_on = False
    if args.l2_mb > 0:
        l2_on = pool.kv_set_l2_residency(args.l2_mb << 20) == B.KV_OK
    N, k = w.N, w.k
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    counts = pool.kv_epoch_counts() if dist_on else None

    def gen_events(e):
        return runner.next_events(e)

    head_obs = [runner.to_device(w.head_observations(0, q).reshape(-1), None) for q in range(len(w.parts))] \
        if args.head_weights else None

    def one_step(e, d_e, d_h, n, ev):
        """Enqueues one full step; ev = (start, selected, D2H done, unpack done, H2D start,
        H2D done) CUDA events.  The promotion's H2D copies run on their own stream and
        overlap the demotion's D2H copies."""
        with torch.cuda.stream(pool.compute):
            ev[0].record(pool.compute)
        if args.head_weights:
            for q in range(len(w.parts)):
                runner.check(pool.kv_head_importance_update(q, head_obs[q], 0.9), "kv_head_importance_update")
        if dist_on:
            runner.check(pool.kv_epoch_events(d_e, d_h, n), "kv_epoch_events")
            with torch.cuda.stream(pool.compute):
                dist.all_reduce(counts)          # 32 int64 counters shared by all pools
            runner.check(pool.kv_epoch_update(e), "kv_epoch_update")
            runner.check(pool.kv_select_victims(k, runner.victims), "kv_select_victims")
        elif args.no_fused:
            runner.check(pool.kv_epoch_score(e, d_e, d_h, n), "kv_epoch_score")
            runner.check(pool.kv_select_victims(k, runner.victims), "kv_select_victims")
        else:
            runner.check(pool.kv_epoch_score_select(e, d_e, d_h, n, k, runner.victims), "kv_epoch_score_select")
        ev[1].record(pool.compute)
        runner.check(runner.demote(), "kv_demote")
        lists = runner.promote_lists(e)
        ev[4].record(pool.copy_h2d)
        for q, lst in enumerate(lists):
            runner.check(pool.kv_promote(q, lst, runner.batch_bytes), "kv_promote")
        runner.check(pool.kv_flush(), "kv_flush")     # the rest of a deferred demotion belongs to the step
        ev[2].record(pool.copy)
        ev[5].record(pool.copy_h2d)
        ev[3].record(pool.compute)
        return sum(len(x) for x in lists), lists

    def between_steps(e):
        runner.check(runner.admit(e), "kv_admit")
        torch.cuda.synchronize(dev)

    def flush_l2(e):
        """Evicts the pool's state from L2 right before a step, on the step's own
        stream: 8 x 256 MiB of writes (each larger than L2).  Queued directly ahead
        of the step, it also means the step does not start on a GPU that has been
        idle while the host drew the trace (the first launch after an idle period
        costs ~30 us extra here, which a serving GPU never sees)."""
        with torch.cuda.stream(pool.compute):
            for i in range(8):
                flush.fill_((e + i) & 0xFF)

    tot = {"ss": 0.0, "dem": 0.0, "pro": 0.0, "all": 0.0, "events": 0, "promoted_bytes": 0}
    ss_steps = []   # score + select of every timed step of this rank, us
    sampler = ClockSampler(local)
    epoch = 0
    launches0 = 0
    for it in range(args.warmup + args.steps):
        timed = it >= args.warmup
        if it == args.warmup:
            if dist_on:
                dist.barrier()
            torch.cuda.synchronize(dev)
            pool.kv_timing_read()                 # discard warm-up launches
            launches0 = pool.kv_get_stats()["kernel_launches"]
            sel0 = pool.kv_selection_stats()
            sampler.start()
        ev_entry, ev_hit = gen_events(epoch)
        d_e, d_h, n = runner.stage_events(ev_entry, ev_hit)
        torch.cuda.synchronize(dev)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
        launches_before = pool.kv_get_stats()["kernel_launches"]
        flush_l2(epoch)
        m, lists = one_step(epoch, d_e, d_h, n, ev)
        torch.cuda.synchronize(dev)
        launches_step = pool.kv_get_stats()["kernel_launches"] - launches_before
        if timed:
            tot["ss"] += ev[0].elapsed_time(ev[1])
            ss_steps.append(round(1e3 * ev[0].elapsed_time(ev[1]), 1))
            tot["dem"] += ev[1].elapsed_time(ev[2])
            tot["pro"] += ev[4].elapsed_time(ev[5])
            tot["all"] += max(ev[0].elapsed_time(ev[2]), ev[0].elapsed_time(ev[3]), ev[0].elapsed_time(ev[5]))
            tot["events"] += n
            tot["promoted_bytes"] += sum(len(l) * p.entry_bytes for l, p in zip(lists, w.parts))
            tot["launches"] = tot.get("launches", 0) + launches_step
        between_steps(epoch)
        epoch += 1
    torch.cuda.synchronize(dev)
    if dist_on:
        dist.barrier()
    clocks = sampler.stop()
    sel1 = pool.kv_selection_stats()
    timing = pool.kv_timing_read()
    status = pool.kv_device_status()
    K = args.steps
    t = torch.tensor([tot["ss"], tot["dem"], tot["pro"], tot["all"]], dtype=torch.float64, device=dev)
    if dist_on:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ss_ms, dem_ms, pro_ms, all_ms = [float(x) / K for x in t.tolist()]

    # ---- end-to-end: host buffers in, host result out, copies inside the timed region -----
    e2e = None
    if not args.no_e2e:
        e2e_steps = max(2, min(K, 5))
        h_vict = torch.empty(max(k, 4), dtype=torch.int32, pin_memory=True)
        wall, h2d_b, d2h_b = 0.0, 0, 0
        for it in range(e2e_steps):
            ev_entry, ev_hit = gen_events(epoch)
            n = int(ev_entry.size)
            h_e = torch.empty(max(n, 4), dtype=torch.int32, pin_memory=True)
            h_h = torch.empty(max(n, 16), dtype=torch.uint8, pin_memory=True)
            h_e[:n] = torch.from_numpy(ev_entry.view(np.int32))
            h_h[:n] = torch.from_numpy(ev_hit)
            d_e = torch.empty_like(h_e, device=dev)
            d_h = torch.empty_like(h_h, device=dev)
            flush_l2(epoch)
            torch.cuda.synchronize(dev)
            if dist_on:
                dist.barrier()
            t0 = time.perf_counter()
            with torch.cuda.stream(pool.compute):
                d_e.copy_(h_e, non_blocking=True)
                d_h.copy_(h_h, non_blocking=True)
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
            m, lists = one_step(epoch, d_e, d_h, n, ev)
            with torch.cuda.stream(pool.compute):
                h_vict[:max(k, 1)].copy_(runner.victims[:max(k, 1)], non_blocking=True)
            torch.cuda.synchronize(dev)
            wall += time.perf_counter() - t0
            h2d_b += n * 5 + sum(len(l) * (p.entry_bytes + 4) for l, p in zip(lists, w.parts))
            d2h_b += k * 4 + sum(c * (p.entry_bytes + 24) for c, p in zip(pool.kv_last_demote_counts(), w.parts))
            between_steps(epoch)
            epoch += 1
        tw = torch.tensor([wall], dtype=torch.float64, device=dev)
        if dist_on:
            dist.all_reduce(tw, op=dist.ReduceOp.MAX)
        e2e = {"value": N * world * e2e_steps / float(tw.item()), "unit": UNIT,
               "scope": "whole epoch (score, select, demote, promote) through the C ABI, events copied in "
                        "from pinned host memory and the victim list read back",
               "h2d_bytes_per_step": h2d_b // e2e_steps, "d2h_bytes_per_step": d2h_b // e2e_steps,
               "steps": e2e_steps, "ms_per_step": 1e3 * float(tw.item()) / e2e_steps}

    # ---- per-call breakdown of scoring + selection (extra epochs after the timed ones) -----
    breakdown = None
    if not args.no_breakdown and not dist_on:
        acc = {"event_reduce": [], "entry_pass": [], "select": []}
        for it in range(3):
            ev_entry, ev_hit = gen_events(epoch)
            d_e, d_h, n = runner.stage_events(ev_entry, ev_hit)
            torch.cuda.synchronize(dev)
            evb = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            flush_l2(epoch)
            evb[0].record(pool.compute)
            runner.check(pool.kv_epoch_events(d_e, d_h, n), "kv_epoch_events")
            evb[1].record(pool.compute)
            runner.check(pool.kv_epoch_update(epoch), "kv_epoch_update")
            evb[2].record(pool.compute)
            runner.check(pool.kv_select_victims(k, runner.victims), "kv_select_victims")
            evb[3].record(pool.compute)
            runner.check(runner.demote(), "kv_demote")
            for q, lst in enumerate(runner.promote_lists(epoch)):
                runner.check(pool.kv_promote(q, lst, runner.batch_bytes), "kv_promote")
            runner.check(pool.kv_flush(), "kv_flush")
            torch.cuda.synchronize(dev)
            for name, i in (("event_reduce", 0), ("entry_pass", 1), ("select", 2)):
                acc[name].append(evb[i].elapsed_time(evb[i + 1]))
            between_steps(epoch)
            epoch += 1
        med = {kk: float(np.median(v)) for kk, v in acc.items()}
        peak_b, kind_b = measured_peaks()
        entry_gbs = 30 * N / (med["entry_pass"] * 1e-3) / 1e9
        breakdown = {"how": "median of 3 extra epochs with the three calls timed one by one (CUDA events, L2 flushed)",
                     "event_reduce_us": 1e3 * med["event_reduce"], "entry_pass_us": 1e3 * med["entry_pass"],
                     "select_us": 1e3 * med["select"],
                     "entry_pass_gbs": entry_gbs, "entry_pass_algorithmic_bytes_per_entry": 30,
                     "entry_pass_frac_of_%s_hbm" % kind_b: entry_gbs / peak_b}

    dedup = None
    if args.dedup and rank == 0:
        dedup = time_dedup(torch, pool, w, B)

    if rank != 0:
        if dist_on:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    eb_bytes = sum(c * p.entry_bytes for c, p in zip(pool.kv_last_demote_counts(), w.parts))
    demoted_per_step = eb_bytes
    promoted_per_step = tot["promoted_bytes"] / K
    pack_gbs = 2 * timing["pack_bytes"] / max(timing["pack_ms"], 1e-9) / 1e6
    unpack_gbs = (2 * timing["unpack_bytes"] / max(timing["unpack_ms"], 1e-9) / 1e6) if timing["unpack_launches"] else None
    ss_bytes = 39 * N + 5 * (tot["events"] / K) + 4 * k
    ss_gbs = ss_bytes / (ss_ms * 1e-3) / 1e9
    fused = not (args.no_fused or dist_on)
    ss_traffic = NCU_SCORE_SELECT_TRAFFIC.get(cfg) if (fused and scale == 1.0 and not args.head_weights
                                                        and args.l2_mb == 48 and l2_on) else None
    tr = NCU_PACK_TRAFFIC_BYTES_PER_PAYLOAD_BYTE
    line = {
        "metric": METRIC, "value": N * world / (ss_ms * 1e-3), "unit": UNIT,
        "value_definition": "N / t(scoring + selection), timed with CUDA events inside full steps; "
                            + ("two calls (kv_epoch_score, kv_select_victims)" if (args.no_fused or dist_on)
                               else "kv_epoch_score_select (event reduction, then entry pass + selection in one kernel)"),
        "n_gpus": world, "steps": K, "warmup": args.warmup, "ms_per_step": all_ms,
        "whole_step_head_blocks_per_s": N * world / (all_ms * 1e-3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": w.name, "pool": cfg, "chosen_because": chosen_because, "n_entries": N, "k": k,
                   "events_per_step": tot["events"] // K, "pool_bytes": sum(p.slab_bytes for p in w.parts),
                   "entry_bytes": [p.entry_bytes for p in w.parts], "batch_bytes": runner.batch_bytes,
                   "deferred_packing": not args.no_deferred_packing,
                   "promote_lists": w.promote_style + ("" if "runs" not in w.promote_style else " of %d slots" % w.max_run),
                   "fused_score_select": not (args.no_fused or dist_on),
                   "l2_residency": ("budget %d MiB: %s in the persisting part of the L2" % (
                       args.l2_mb, "touch counts" if 4 * N <= (args.l2_mb << 20) else "pair bytes")) if l2_on else "off",
                   "head_weights": bool(args.head_weights),
                   "ring_slots": [p.ring_slots for p in w.parts], "scale": scale,
                   "parallelism": "1 pool per GPU" + (", 256-byte all-reduce of pair counters" if dist_on else ""),
                   "l2": "flushed before every step: 8 x 256 MiB written on the step's stream (and >1 GB of "
                         "fresh blocks admitted between steps)"},
        "phases": {
            "score_select_ms": ss_ms,
            "score_select_us_per_step": ss_steps,
            "score_select_effective_gbs": ss_gbs,
            "demote_ms": dem_ms, "demote_gbs": demoted_per_step / (dem_ms * 1e-3) / 1e9,
            "promote_ms": pro_ms, "promote_gbs": promoted_per_step / max(pro_ms * 1e-3, 1e-12) / 1e9,
            "pack_kernel_gbs": pack_gbs, "pack_kernel_frac_of_%s_hbm" % peak_kind: pack_gbs / peak,
            "unpack_kernel_gbs": unpack_gbs,
            "unpack_kernel_frac_of_%s_hbm" % peak_kind: (unpack_gbs / peak) if unpack_gbs else None,
            "pack_launches": timing["pack_launches"], "unpack_launches": timing["unpack_launches"],
            "gather_launches": timing["gather_launches"],
            "gather_kernel_gbs_over_the_host_link": (timing["gather_bytes"] / max(timing["gather_ms"], 1e-9) / 1e6
                                                     if timing["gather_launches"] else None),
        },
        "hostlink": link,
        "roofline": {"kernel": ("event_reduce_kernel + select_persistent_kernel<true>" if fused else
                                "event_reduce_kernel + entry_update_kernel + select_persistent_kernel<false>")
                               + " (the scoring + selection pass that `value` times)",
                     "bound": "hbm", "achieved": ss_gbs, "peak": peak, "peak_kind": "of " + peak_kind, "unit": "GB/s",
                     "frac": ss_gbs / peak, "traffic": ss_traffic,
                     "algorithmic_bytes_per_launch": ss_bytes,
                     "algorithmic_bytes": "39 B/entry (30 scoring + 9 selection) + 5 B/event + 4 B/victim",
                     "launch_us": 1e3 * ss_ms,
                     "launch_us_median": float(np.median(ss_steps)) if ss_steps else None,
                     "selection_hints": {"selections": sel1["selections"] - sel0["selections"],
                                         "hits": sel1["hint_hits"] - sel0["hint_hits"],
                                         "misses": sel1["hint_misses"] - sel0["hint_misses"],
                                         "thread_blocks_that_reread_their_keys": sel1["reread_ctas"] - sel0["reread_ctas"]}},
        "roofline_pack": {"kernel": PACK_KERNEL_NAME, "bound": "hbm", "achieved": pack_gbs, "peak": peak,
                          "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": pack_gbs / peak,
                          "traffic": tr * timing["pack_bytes"] / max(timing["pack_launches"], 1),
                          "algorithmic_bytes_per_launch": 2 * timing["pack_bytes"] / max(timing["pack_launches"], 1)},
        "clocks": clocks,
        "gpu_launches": tot.get("launches", 0),
        "device_status": status,
    }
    if link:
        line["phases"]["demote_frac_of_d2h_link"] = line["phases"]["demote_gbs"] / link["d2h_gbs"]
        line["phases"]["promote_frac_of_h2d_link"] = line["phases"]["promote_gbs"] / link["h2d_gbs"]
        # the promotion's copies run while the demotion's do: the link's rate per direction with both busy
        line["phases"]["promote_frac_of_link_with_both_directions_busy"] = \
            line["phases"]["promote_gbs"] / link["bidir_gbs_per_dir"]
    if dedup:
        line["phases"].update(dedup)
    if breakdown:
        line["phases"]["score_select_breakdown"] = breakdown
    if e2e:
        line["e2e"] = e2e
    if not args.no_cpu_baseline:
        n_ep = 6
        # (a workload of its own: the trace generators keep session state from epoch to epoch)
        w_cpu = W.config(cfg, scale=scale, ring_slots=args.ring_slots, tiny_entries=args.tiny_entries)
        t_ss, t_all, done = oracle_epochs(w_cpu, n_ep, warm=1)
        mv = oracle_movement(W, cfg)
        line["cpu_baseline"] = {
            "value": N * done / t_ss, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": "%d epochs of the same pool (N=%d, k=%d) in metadata mode, score+select timed; host has %d cores"
                      % (done, N, k, os.cpu_count() or 0),
            "ms_per_epoch_score_select": 1e3 * t_ss / done,
            "whole_epoch_head_blocks_per_s": N * done / t_all,
            "movement": {"demote_gbs": mv["demote_gbs"], "promote_gbs": mv["promote_gbs"],
                         "sample": "%d epochs of the same pool scaled by %.4g (%.2f GiB of blocks) in payload mode: "
                                   "memcpy-based demotion and promotion, 1 thread"
                                   % (mv["epochs"], mv["scale"], mv["pool_bytes"] / 2**30)}}
    print(json.dumps(line))
    runner.close()
    if dist_on:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
