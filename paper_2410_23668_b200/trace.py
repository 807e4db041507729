"""Stage timeline of the looped decoder kernel, read through kl_set_trace.

    python -m paper_2410_23668_b200.trace [--workload llama31_8b_b1_ctx4096] [--warm 5] [--greedy]

Runs a few warm-up steps, then one traced decode step (kl_decode_step: the decoder kernel; with --greedy
kl_decode_greedy: the one-launch-per-token kernel, whose decoder layers take the same stamps), and prints per stage of a layer the median / maximum /
minimum over the CTAs of the time between consecutive stamps (microseconds, averaged over layers 1..L-1), the
sub-steps of the attention block for the CTAs that own a split-K unit, and the per-chunk statistics of CTA 0.
Stamp meanings are listed next to kl_set_trace in include/kl.h.  Tracing costs a few percent: use bench.py for
throughput and this for where the time goes.
"""
from __future__ import annotations

import argparse
import sys
from pathlib import Path

import numpy as np
import torch

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

from paper_2410_23668_b200 import inputs as gen  # noqa: E402

SEQ = [(0, "layer entered"), (1, "input normalised"), (2, "QKV rows done"), (4, "attention block done"),
       (6, "attention output loaded"), (7, "O rows done"), (9, "x' normalised"), (10, "gate/up rows done"),
       (12, "h counter passed"), (13, "down rows done")]
ATTN = [(2, 14, "QKV done -> q/k/v polled, rotated"), (14, 15, "-> ring chunks consumed (warp 0)"),
        (15, 3, "-> partial result written"), (3, 5, "-> slice loads complete (thread 0)"), (5, 4, "-> block done")]


def main() -> None:
    import bench  # the workloads and the model builder live there
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="llama31_8b_b1_ctx4096", choices=sorted(bench.WORKLOADS))
    ap.add_argument("--warm", type=int, default=5)
    ap.add_argument("--greedy", action="store_true", help="trace the one-launch-per-token kernel (kl_decode_greedy)")
    args = ap.parse_args()
    shape, batch, context, _ = bench.WORKLOADS[args.workload]
    assert batch == 1, "the timeline is read for one sequence"
    dec, cache, _ = bench.build_model(shape, batch, context, args.warm + 8)
    P, L, NS = dec.kl_set_trace(None)
    nchunk_rows = 8192
    buf = torch.zeros(P * L * NS + nchunk_rows * 4, dtype=torch.int64, device="cuda")
    tok = gen.make_tokens(shape, batch, 0, device="cuda")
    pos = torch.full((batch,), context, dtype=torch.int32, device="cuda")
    logits = torch.empty(batch, shape.vocab, device="cuda")
    for _ in range(args.warm):
        dec.kl_decode_step(tok, pos, cache, logits, batch)
        dec.kl_argmax_advance(logits, tok, pos, batch)
    if args.greedy:
        dec.kl_decode_greedy(tok, pos, cache, logits, batch, True)
    dec.kl_set_trace(buf)
    if args.greedy:
        dec.kl_decode_greedy(tok, pos, cache, logits, batch, False)
    else:
        dec.kl_decode_step(tok, pos, cache, logits, batch)
    torch.cuda.synchronize()
    status = dec.kl_last_status()
    raw = buf.cpu().numpy()
    dec.kl_set_trace(None)
    dec.close()
    if status != 0:
        raise SystemExit(f"device status {status}")
    stamps = raw[:P * L * NS].reshape(P, L, NS).astype(np.float64)
    t0 = stamps[:, 0, 0].min()
    tt = (stamps - t0) / 1e3
    lay = slice(1, L) if L > 1 else slice(0, 1)
    print(f"workload {args.workload}: {P} CTAs, {L} layers; microseconds")
    print(f"{'segment':58s} {'median':>8s} {'max':>8s} {'min':>8s}")
    total = 0.0
    for (a, na), (b, nb) in zip(SEQ[:-1], SEQ[1:]):
        d = tt[:, lay, b] - tt[:, lay, a]
        med = float(np.median(d, axis=0).mean())
        total += med
        print(f"{na + ' -> ' + nb:58s} {med:8.2f} {d.max(axis=0).mean():8.2f} {d.min(axis=0).mean():8.2f}")
    if L > 2:
        d = tt[:, 2:, 0] - tt[:, 1:-1, 13]
        med = float(np.median(d, axis=0).mean())
        total += med
        print(f"{'down rows done -> next layer entered':58s} {med:8.2f}")
    print(f"{'sum of medians':58s} {total:8.2f}")
    per_layer = [float(tt[:, l, 13].max() - tt[:, l, 0].min()) for l in range(L)]
    print("layer time, first entry to last exit:", " ".join(f"{x:.1f}" for x in per_layer[:8]), "...")
    act = tt[:, min(1, L - 1), 14] > 0
    print(f"attention block, {int(act.sum())} CTAs with a split-K unit:")
    for a, b, name in ATTN:
        d = tt[act][:, lay, b] - tt[act][:, lay, a]
        print(f"  {name:56s} {np.median(d):8.2f} {d.max():8.2f} {d.min():8.2f}")
    ch = (raw[P * L * NS:].reshape(nchunk_rows, 4).astype(np.float64) - t0) / 1e3
    ok = raw[P * L * NS:].reshape(nchunk_rows, 4)[:, 3] > 0
    l = min(2, L - 1)
    print(f"ring chunks of CTA 0 in layer {l}: stage, chunks, issue->landed, landed->dot done, dot done->emitted, GB/s of the CTA")
    for name, a, b in (("QKV", 1, 2), ("O", 6, 7), ("gate/up", 9, 10), ("down", 12, 13)):
        lo, hi = tt[0, l, a], tt[0, l, b]
        sel = [n for n in np.nonzero(ok)[0] if lo <= ch[n][3] <= hi]
        if not sel:
            continue
        il = np.array([ch[n][2] - ch[n][0] for n in sel])
        lc = np.array([ch[n][1] - ch[n][2] for n in sel])
        cd = np.array([ch[n][3] - ch[n][1] for n in sel])
        print(f"  {name:8s} {len(sel):4d} {np.median(il):7.2f} {np.median(lc):7.2f} {np.median(cd):7.2f} "
              f"{len(sel) * 16384 / max(hi - lo, 1e-9) / 1e3:8.1f}")


if __name__ == "__main__":
    main()
