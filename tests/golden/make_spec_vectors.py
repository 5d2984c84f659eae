"""Writes tests/golden/sbw_spec_v1_vectors.txt from the big-integer restatement in oracle/py_ref.

Run from the repository root:  python tests/golden/make_spec_vectors.py
Only ``oracle/`` is called; nothing from the CUDA library.  The file pins the frozen reading
("SBW-spec v1") of the hashes the paper names in Sections 2.2 and 2.3 without printing them.
"""
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent.parent
sys.path.insert(0, str(ROOT))
from oracle import py_ref as R  # noqa: E402

KEY = 0x5EED
lines = ["# SBW-spec v1 known answers (Section 2.2: Philox 4x32-10; Section 2.3: Jenkins hash;",
         "# Table 12: additive / anchored-minhash PRFs).  Written by make_spec_vectors.py."]
for a in (0, 1, 2, 0x5EED, 128255, 151935, 0xFFFFFFFF):
    lines.append(f"jenkins {a:#x} {R.jenkins(a):#010x}")
for ctr, key in (((0, 0, 0, 0), (0, 0)),
                 ((0xFFFFFFFF,) * 4, (0xFFFFFFFF,) * 2),
                 ((1, 0, 0, 0), (KEY, 0)),
                 ((0, 0, 0, 0), (KEY, 0)),
                 ((12345, 0, 0, 0), (KEY, 0)),
                 ((0x243F6A88, 0x85A308D3, 0x13198A2E, 0x03707344), (0xA4093822, 0x299F31D0))):
    out = R.philox4x32_10(ctr, key)
    lines.append("philox " + " ".join(f"{x:#x}" for x in ctr) + " | " +
                 " ".join(f"{x:#x}" for x in key) + " | " + " ".join(f"{x:08x}" for x in out))
lines.append(f"seed_context {KEY:#x} 7 {R.seed_context(KEY, [7]):#x}")
for v in range(4):
    lines.append(f"seed_selfsalt {KEY:#x} 7 {v} {R.seed_selfsalt(KEY, [7], v):#018x}")
for v in range(4):
    r = R.seed_context(KEY, [7])
    x = R.philox4x32_10((v, 0, 0, 0), (r & R.M32, r >> 32))[0]
    lines.append(f"word0_context {KEY:#x} 7 {v} {x:08x}")
lines.append("green_context 0.25 " + R.green_bits(KEY, [7], 0.25, "context", range(16)))
lines.append("green_selfsalt 0.25 " + R.green_bits(KEY, [7], 0.25, "selfsalt", range(16)))
for V, gamma, scheme in ((32000, 0.25, "context"), (128256, 0.5, "context"), (32000, 0.25, "selfsalt")):
    n = R.green_bits(KEY, [12345], gamma, scheme, range(V)).count("1")
    lines.append(f"green_count {scheme} {V} {gamma} 12345 {n}")
(Path(__file__).resolve().parent / "sbw_spec_v1_vectors.txt").write_text("\n".join(lines) + "\n")
print("\n".join(lines))
