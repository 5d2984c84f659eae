"""The stored known answers of the sampler part of SBW-spec v1 (tests/golden/, written by
make_sampler_vectors.py from the oracle alone): the oracle must still reproduce them -- a change
of its arithmetic has to be deliberate -- and, on a GPU, the CUDA library must reproduce the ids."""
import importlib.util
import re
from pathlib import Path

import numpy as np
import pytest
import torch

GOLDEN = Path(__file__).resolve().parent / "golden"


def _script():
    spec = importlib.util.spec_from_file_location("make_sampler_vectors", GOLDEN / "make_sampler_vectors.py")
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_oracle_reproduces_the_stored_sampler_vectors():
    stored = (GOLDEN / "sbw_spec_v1_sampler_vectors.txt").read_text().splitlines()
    assert _script().lines() == stored
    assert sum(l.startswith("log ") for l in stored) == 8 and sum(l.startswith("filtered ") for l in stored) == 6
    # two of the stored logarithms by hand: L(1) = 0 exactly, L(2) = LN2_HI + LN2_LO rounded = fl(ln 2)
    assert "log 0x1.0000000000000p+0 0x0.0p+0" in stored
    assert f"log 0x1.0000000000000p+1 {float(np.float32(np.log(2.0))).hex()}" in stored


@pytest.mark.gpu
def test_cuda_library_reproduces_the_stored_ids():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2609_03844_b200 as sbw

    dev = torch.device("cuda:0")
    mod = _script()
    x = torch.from_numpy(mod.table(2, 257)).to(dev)
    ctx = torch.tensor([[7], [9]], dtype=torch.int32, device=dev)
    ids = torch.empty(2, dtype=torch.int32, device=dev)
    kept = torch.empty(2, dtype=torch.int32, device=dev)
    ws = torch.empty(max(sbw.sbw_sample_workspace_bytes(2, 257), 256), dtype=torch.uint8, device=dev)
    wsf = torch.empty(max(sbw.sbw_sample_filtered_workspace_bytes(torch.float32, 2, 257), 256), dtype=torch.uint8,
                      device=dev)
    for line in (GOLDEN / "sbw_spec_v1_sampler_vectors.txt").read_text().splitlines():
        if line.startswith("sample "):
            scheme = int(re.search(r"scheme=(\d)", line).group(1))
            want = [tuple(map(int, p.split(","))) for p in line.split()[2:]]
            for step, w in enumerate(want):
                sbw.sbw_bias_sample(x, ctx, mod.KEY, 0.25, 2.0, scheme, 0.7, 0xC4, step, ids, ws)
                assert tuple(ids.cpu().tolist()) == w, line
        elif line.startswith("filtered "):
            scheme = int(re.search(r"scheme=(\d)", line).group(1))
            top_k = int(re.search(r"top_k=(\d+)", line).group(1))
            top_p = float(re.search(r"top_p=([0-9.]+)", line).group(1))
            want_kept = [int(v) for v in re.search(r"kept=\[([0-9, ]+)\]", line).group(1).split(",")]
            want = [tuple(map(int, p.split(","))) for p in line.split("] ")[1].split()]
            for step, w in enumerate(want):
                sbw.sbw_bias_sample_filtered(x, ctx, mod.KEY, 0.25, 2.0, scheme, 0.7, top_k, top_p, 0xC4, step, ids,
                                             wsf, out_kept=kept)
                assert tuple(ids.cpu().tolist()) == w, line
                if step == 0:
                    assert kept.cpu().tolist() == want_kept, line
