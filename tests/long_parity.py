"""Full-length closed-loop parity runs: the CUDA library against the CPU oracle over a whole workload.

The pytest suite compares windows of a few steps at the large shapes, so that it ends in minutes; this
script runs a workload for as many steps as asked (its full length by default), comparing every emitted
token and every drafted tree of every step and, at the end (and every --check-every steps), the sequence
state and the whole N-gram table.  It needs a GPU and the built oracle; one JSON line per run.

    python tests/long_parity.py --workload cfg3                 # all 8,192 steps
    python tests/long_parity.py --workload cfg5 --steps 128 --peak-mode p80

Every run appends its JSON line to --record (tests/parity_runs.jsonl by default), the tracked record of these runs.
"""
import argparse
import json
import os
import sys
import time

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from paper_2506_04708_b200 import inputs  # noqa: E402
from tests import harness  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="cfg1", choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--steps", type=int, default=0, help="0 = the workload's full length")
    ap.add_argument("--peak-mode", default="add8", choices=["add8", "p80"])
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--check-every", type=int, default=0, help="also compare state and table every so many steps")
    ap.add_argument("--deterministic", action="store_true")
    ap.add_argument("--record", default=os.path.join(os.path.dirname(os.path.abspath(__file__)), "parity_runs.jsonl"),
                    help="file the run's JSON line is appended to")
    args = ap.parse_args()

    w = inputs.WORKLOADS[args.workload]
    steps = args.steps or w.steps
    w = inputs.scaled(w, steps=steps)
    big = w.B * w.N * w.V > 1 << 21  # large shapes: logits made on the device, copied to the host for the oracle
    t0 = time.time()
    loop = harness.ClosedLoop(w, seed=args.seed, peak_mode=args.peak_mode, device_logits=big,
                              deterministic=args.deterministic)
    checks = []
    try:
        for s in range(steps):
            loop.step()
            if (s + 1) % max(1, steps // 16) == 0:  # progress, so that a run cut short still says how far it got
                print(json.dumps({"progress": s + 1, "hard_mismatches": len(loop.hard), "tolerated_low_margin": loop.tolerated,
                                  "seconds": round(time.time() - t0, 1)}), file=sys.stderr, flush=True)
            if args.check_every and (s + 1) % args.check_every == 0 and s + 1 < steps:
                checks.append(len(loop.check_state_and_table()))
        final = loop.check_state_and_table()
        st = loop.gpu.stats()
        contexts = len(loop.orc.table())
    finally:
        loop.close()
    out = {
        "workload": args.workload, "steps": steps, "peak_mode": args.peak_mode, "seed": args.seed,
        "drafting": "deterministic" if args.deterministic else "stochastic",
        "rows_compared": steps * w.B * w.N, "emitted_tokens": loop.emitted_total,
        "acceptance_length": loop.emitted_total / (steps * w.B),
        "hard_mismatches": len(loop.hard), "tolerated_low_margin": loop.tolerated, "tolerated_by": loop.tolerated_by,
        "state_and_table_differences": len(final), "intermediate_checks": checks,
        "table_contexts": contexts, "drops": st["drops"], "bad_tokens": st["bad_tokens"],
        "wait_timeouts": st["wait_timeouts"], "max_probe": st["max_probe_seen"], "seconds": round(time.time() - t0, 1),
    }
    print(json.dumps(out), flush=True)
    with open(args.record, "a") as f:
        f.write(json.dumps(out) + "\n")
    ok = not loop.hard and not final and not any(checks) and st["drops"] == 0 and st["wait_timeouts"] == 0
    sys.exit(0 if ok else 1)


if __name__ == "__main__":
    main()
