"""Sweeps the victim fraction k and the demote/promote batch size on one pool.

    python -m paper_2604_26968_b200.sweep POOL SCALE K_FRACS BATCHES_MIB
    e.g. python -m paper_2604_26968_b200.sweep 5 0.25 0.01,0.05,0.10,0.25 1,4,16,64,256,1024

Prints a markdown table: per (k, batch) the event-timed score+select time, the
demote (D2H) and promote (H2D, overlapped with the D2H) rates over the host
link, the event-timed pack/unpack kernel rates and the whole-step time.
"""
import gc
import sys


def sweep(cfg, scale, kfracs, batches_mib, out=sys.stdout):
    import torch

    from . import workloads as W
    from .harness import EpochRunner

    dev = torch.device("cuda:0")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    print("| pool | N | k frac | batch MiB | score+select us | G head-blocks/s | demote GB/s | promote GB/s "
          "| pack GB/s | unpack GB/s | step ms |", file=out)
    print("|---|---|---|---|---|---|---|---|---|---|---|", file=out)
    for kf in kfracs:
        w = W.config(cfg, scale=scale)
        w.evict_frac = kf
        w.epochs = 24
        for p in w.parts:
            if cfg == 5:   # rings sized to the sweep's k, with room for older entries
                p.ring_slots = min(p.n_entries, int(1.6 * w.k)) + 64
        r = EpochRunner(w, batch_bytes=max(batches_mib) << 20, fill_pattern=True, host_meta=True)
        p = r.pool
        p.kv_timing_enable(True)
        p.kv_set_deferred_packing(True)
        e = 0
        for _ in range(2):
            ev_entry, ev_hit = r.next_events(e)
            d_e, d_h, n = r.stage_events(ev_entry, ev_hit)
            r.step(e, d_e, d_h, n)
            e += 1
        for mb in batches_mib:
            r.batch_bytes = mb << 20
            acc = dict(ss=0.0, dem=0.0, pro=0.0, allms=0.0, dbytes=0, pbytes=0)
            p.sync()
            p.kv_timing_read()
            steps = 2
            for _ in range(steps):
                ev_entry, ev_hit = r.next_events(e)
                d_e, d_h, n = r.stage_events(ev_entry, ev_hit)
                torch.cuda.synchronize()
                with torch.cuda.stream(p.compute):
                    for i in range(8):
                        flush.fill_(i)
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
                ev[0].record(p.compute)
                r.check(p.kv_epoch_score_select(e, d_e, d_h, n, r.k, r.victims), "score+select")
                ev[1].record(p.compute)
                r.check(r.demote(), "demote")
                lists = r.promote_lists(e)
                ev[4].record(p.copy_h2d)
                for q, lst in enumerate(lists):
                    r.check(p.kv_promote(q, lst, r.batch_bytes), "promote")
                r.check(p.kv_flush(), "flush")
                ev[2].record(p.copy)
                ev[5].record(p.copy_h2d)
                ev[3].record(p.compute)
                torch.cuda.synchronize()
                acc["ss"] += ev[0].elapsed_time(ev[1])
                acc["dem"] += ev[1].elapsed_time(ev[2])
                acc["pro"] += ev[4].elapsed_time(ev[5])
                acc["allms"] += max(ev[0].elapsed_time(ev[2]), ev[0].elapsed_time(ev[3]), ev[0].elapsed_time(ev[5]))
                acc["dbytes"] += sum(c * pp.entry_bytes for c, pp in zip(p.kv_last_demote_counts(), w.parts))
                acc["pbytes"] += sum(len(l) * pp.entry_bytes for l, pp in zip(lists, w.parts))
                r.check(r.admit(e), "admit")
                e += 1
            t = p.kv_timing_read()
            print("| %d | %d | %.2f | %d | %.1f | %.1f | %.1f | %.1f | %.0f | %.0f | %.2f |" % (
                cfg, w.N, kf, mb, 1e3 * acc["ss"] / steps, w.N / (acc["ss"] / steps * 1e-3) / 1e9,
                acc["dbytes"] / acc["dem"] / 1e6, acc["pbytes"] / max(acc["pro"], 1e-9) / 1e6,
                2 * t["pack_bytes"] / max(t["pack_ms"], 1e-9) / 1e6,
                2 * t["unpack_bytes"] / max(t["unpack_ms"], 1e-9) / 1e6, acc["allms"] / steps), file=out, flush=True)
        assert p.kv_device_status() == 0
        r.close()
        del r, p
        gc.collect()
        torch.cuda.empty_cache()


def main(argv):
    if len(argv) != 5:
        raise SystemExit(__doc__)
    sweep(int(argv[1]), float(argv[2]), [float(x) for x in argv[3].split(",")],
          [int(x) for x in argv[4].split(",")])


if __name__ == "__main__":
    main(sys.argv)
