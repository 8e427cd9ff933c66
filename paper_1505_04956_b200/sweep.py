"""Worker / communication sweep and the communication ablations on one GPU.

For every point (W, c, Parzen window on/off, rows per message) of a grid it runs free-running passes of
a workload through the library and prints one JSON line: samples/s of the last pass (CUDA events), the
quantisation error E(w) of worker 0's state and of the mean state (Eq. 8), the mean distance of worker 0's
centres to the generator's centres under a greedy pairing (Section 5.4), and the message counters
(sent, received, accepted = "good", overwritten) summed over the workers.  c = 0 is the silent mode
(no communication at all), --no-parzen accepts every non-empty message.

    python -m paper_1505_04956_b200.sweep --workload sweep --workers 148,592,2368 --comm-interval 0,1,10,100
"""
import argparse
import json


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="sweep")
    ap.add_argument("--rows", type=int, default=0)
    ap.add_argument("--workers", default="", help="comma-separated W values (default: the workload's)")
    ap.add_argument("--comm-interval", default="", help="comma-separated c values (default: the workload's)")
    ap.add_argument("--parzen", default="1", help="comma-separated 1/0")
    ap.add_argument("--partial-rows", default="0", help="comma-separated rows per message, 0 = whole state")
    ap.add_argument("--passes", type=int, default=2)
    args = ap.parse_args()

    import torch
    import paper_1505_04956_b200 as pkg
    from paper_1505_04956_b200 import inputs, metrics

    pkg.load()
    base = inputs.WORKLOADS[args.workload]
    if args.rows:
        base = base.scaled(N=args.rows)
    X, mu = inputs.make_samples(base, device="cuda")
    mu = mu.cpu().numpy()
    w0 = inputs.initial_centres(base, X)
    ints = lambda text, default: [int(v) for v in text.split(",")] if text else [default]
    for W in ints(args.workers, base.W):
        for c in ints(args.comm_interval, base.comm_interval):
            for parzen in ints(args.parzen, 1):
                for rows in ints(args.partial_rows, 0):
                    wl = base.scaled(W=W, comm_interval=c)
                    cfg = pkg.make_config(N=wl.N, d=wl.d, k=wl.k, W=wl.W, b=wl.b, eps=wl.eps, comm_interval=c,
                                          fanout=wl.fanout, seed=wl.seed, parzen=parzen, partial_rows=rows)
                    ctx = pkg.Asgd(cfg, X, w0)
                    steps = wl.B
                    for _ in range(args.passes - 1):
                        ctx.run(steps)
                    ctx.sync()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    ctx.run(steps)
                    e1.record()
                    torch.cuda.synchronize()
                    ctx.sync()
                    ms = e0.elapsed_time(e1)
                    msgs = {"sent": 0, "received": 0, "accepted": 0, "overwritten": 0}
                    for i in range(wl.W):
                        st = ctx.get_stats(i)
                        for key in msgs:
                            msgs[key] += st[key]
                    print(json.dumps({
                        "workload": wl.name, "W": W, "comm_interval": c, "parzen": parzen, "partial_rows": rows,
                        "passes": args.passes, "steps_per_worker_per_pass": steps, "kernel": ctx.path_name(),
                        "ms_last_pass": ms, "samples_per_s": wl.W * steps * wl.b / (ms * 1e-3),
                        "E_worker0": ctx.eval(0), "E_mean_state": ctx.eval(-1),
                        "generator_centre_error_worker0": metrics.generator_centre_error(mu, ctx.get_state(0).cpu().numpy())[0],
                        "messages": msgs}), flush=True)
                    ctx.destroy()


if __name__ == "__main__":
    main()
