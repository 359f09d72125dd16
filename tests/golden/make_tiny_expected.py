"""Writes tests/golden/tiny_stream_expected.txt from the CPU oracle alone (never from the CUDA path).

The tiny workload (1 layer, batch 1, 2 heads, head_dim 64, 16 tokens per frame, 3-frame chunks, 6-frame window,
no sink, 4 chunks streamed with evict/append) is run through oracle.rolling_attn; per chunk a few scalar
summaries of O, LSE, dQ, dK, dV are stored with 12 significant digits.  The file guards the oracle against
accidental changes of its arithmetic: tests/test_oracle_pins.py recomputes and compares.

    python tests/golden/make_tiny_expected.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import rolling_attn as orc  # noqa: E402
from paper_2603_17051_b200 import synth  # noqa: E402  (seeded inputs only)


def tiny_stream_summaries():
    w = synth.TINY
    model = orc.RollingKVCache(w.sink_frames, w.window_frames)
    M = w.chunk_tokens
    rows = []
    for n in range(4):
        over = model.held() - (w.sink_frames + w.window_frames - w.chunk_frames)
        if over > 0:
            model.evict(over)
        bits = [synth.normal_bf16(synth.tensor_seed(1, 10 * n + i), (w.batch, M, w.heads, w.head_dim)) for i in range(4)]
        q, kc, vc, do = (orc.bf16_bits_to_f64(x) for x in bits)
        kx, vx = model.export()
        kx = None if kx is None else orc.bf16_bits_to_f64(kx)
        vx = None if vx is None else orc.bf16_bits_to_f64(vx)
        o, lse = orc.chunk_attn_fwd(q, kx, vx, kc, vc, w.scale)
        dq, dk, dv = orc.chunk_attn_bwd(q, kx, vx, kc, vc, do, w.scale)
        for name, t in (("O", o), ("LSE", lse), ("dQ", dq), ("dK", dk), ("dV", dv)):
            rows.append((n, name, float(t.sum()), float(np.abs(t).sum()), float(t.reshape(-1)[7]), float(t.reshape(-1)[-3])))
        model.append(bits[1], bits[2], w.tokens_per_frame)
    return rows


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_stream_expected.txt")
    with open(path, "w") as f:
        f.write("# chunk tensor sum abs_sum element[7] element[-3]   (fp64 oracle, tiny workload; see make_tiny_expected.py)\n")
        for n, name, s, a, e7, e3 in tiny_stream_summaries():
            f.write("%d %s %.12e %.12e %.12e %.12e\n" % (n, name, s, a, e7, e3))
    print("wrote", path)
