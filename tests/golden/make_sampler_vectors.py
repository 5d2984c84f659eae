"""Writes tests/golden/sbw_spec_v1_sampler_vectors.txt: known answers of the parts of "SBW-spec v1"
that this library specifies itself because the paper leaves sampling to the serving engine
(Section 5.1) -- the fixed fp32 logarithm, the Gumbel stream, the integer softmax weights of the
top-p cut, and sampled ids on a small closed-form logits table.

Run from the repository root:  python tests/golden/make_sampler_vectors.py
Only ``oracle/`` is called; nothing from the CUDA library.
"""
import sys
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent.parent.parent
sys.path.insert(0, str(ROOT))
import oracle  # noqa: E402

KEY = 0x5EED


def table(B, V):
    """Closed-form logits: no random generator involved."""
    j = np.arange(V, dtype=np.int64)
    rows = [(((j * 37 + 11 * b) % 101) / 10.0 - 5.0) for b in range(B)]
    return np.asarray(rows, dtype=np.float32)


def lines():
    out = ["# SBW-spec v1, sampler part (specified by this library; the paper leaves sampling to the serving",
           "# engine, Section 5.1, and samples with temperature 0.7 / top_p 0.8 in Appendix F).",
           "# Written by make_sampler_vectors.py from the CPU oracle."]
    for x in (0.5, 1.0, 1.5, 2.0, 3.1415927, 1e-3, 6.0e-8, 15.9424):
        x32 = float(np.float32(x))
        out.append(f"log {x32.hex()} {oracle.log32(x32).hex()}")
    for seed, step, row, v in ((0xC4, 0, 0, 0), (0xC4, 0, 0, 1), (0xC4, 1, 0, 0), (0xC4, 0, 3, 128255),
                               (1 << 40, 1 << 33, 1023, 151935)):
        out.append(f"gumbel {seed:#x} {step:#x} {row} {v} {oracle.gumbel_uniform(seed, step, row, v).hex()} "
                   f"{oracle.gumbel(seed, step, row, v).hex()}")
    c = float(np.float32(1.4426950408889634 / 0.7))
    for l, m in ((0.0, 0.0), (-0.25, 0.0), (3.5, 7.25), (-12.0, 7.25), (-12.625, 7.25), (-13.0, 7.25)):
        out.append(f"weight {l} {m} {c.hex()} {oracle.nucleus_weight(l, m, False, c)}")
    x = table(2, 257)
    ctx = np.array([[7], [9]], dtype=np.int32)
    for scheme in (0, 1):
        ids = [oracle.bias_sample(x, 257, ctx, KEY, 0.25, 2.0, scheme, 0.7, 0xC4, step)["tokens"].tolist()
               for step in range(4)]
        out.append(f"sample scheme={scheme} " + " ".join(f"{a},{b}" for a, b in ids))
        for top_k, top_p in ((0, 0.8), (40, 1.0), (10, 0.5)):
            r = [oracle.bias_sample_filtered(x, 257, ctx, KEY, 0.25, 2.0, scheme, 0.7, top_k, top_p, 0xC4, step)
                 for step in range(4)]
            out.append(f"filtered scheme={scheme} top_k={top_k} top_p={top_p} kept={r[0]['kept'].tolist()} " +
                       " ".join(f"{q['tokens'][0]},{q['tokens'][1]}" for q in r))
    return out


if __name__ == "__main__":
    text = "\n".join(lines()) + "\n"
    (Path(__file__).resolve().parent / "sbw_spec_v1_sampler_vectors.txt").write_text(text)
    print(text, end="")
