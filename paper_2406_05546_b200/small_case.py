"""A reduced run of the stateless workload for profiling: a few ticks, an outage that buffers a few
GB of gradients, and the catch-up replay.  Sized so that a profiler's multi-pass capture of one
kernel ends by itself (the queue is larger than L2 but only a few GB).

    python -m paper_2406_05546_b200.small_case [--workers 16] [--batch 64] [--down-ticks 50] [--ticks 3]
"""
import argparse

import numpy as np


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workers", type=int, default=16)
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--ticks", type=int, default=3)
    ap.add_argument("--down-ticks", type=int, default=50)
    ap.add_argument("--precision", type=int, default=0)
    args = ap.parse_args()
    import torch
    from . import harness, ps, schedules, synth
    s = schedules.Schedule("small", W=args.workers, b=args.batch, mode=schedules.REPLAY,
                           ticks=2 * args.ticks + args.down_ticks, external_store=True,
                           kill_at=args.ticks, recover_at=args.ticks + args.down_ticks, recover_by="restore",
                           replay_scale=1.0 / max(1, args.down_ticks))
    px, py = synth.image_pool(8192, seed=0)
    srv = harness.make_server(s, synth.init_params(1), precision=args.precision)
    log = harness.run(s, srv, px, py)
    torch.cuda.synchronize()
    st = srv.ps_stats()
    replay = log[s.recover_at]["apply"]
    theta = srv.ps_export_params()[0]
    assert np.isfinite(theta).all()
    print(f"small case: W={s.W} b={s.b}, {len(log)} ticks, replayed {replay['applied']} gradients "
          f"({replay['applied'] * ps.P * 4 / 1e9:.2f} GB), version {st['version']}, launches {st['kernel_launches']}")
    srv.close()


if __name__ == "__main__":
    main()
