"""sbw_bias_sample_noalloc against sbw_bias_sample and against the oracle.

Some callers of this library cannot allocate device memory -- a logits processor running inside
a serving engine that handed the whole GPU to its cache pool, a component under a fixed memory
budget -- so one entry point takes its scratch from a fixed array inside the library.  This file
checks, through the C ABI, that it returns what the workspace-taking entry point and the CPU
oracle return, on calls in a row of different shapes (the array keeps an earlier call's contents
when the next one starts, also when the next one has more rows), and that it refuses batches
beyond its stated capacity.  The file name sorts last so that a run that stops
at the first failure has already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2609_03844_b200 as sbw
from paper_2609_03844_b200 import binding, inputs
from gpu_util import KEY, require_gpu

REL = 1e-6


def _both(dev, B, V, dtype, scheme, step, seed, oracle):
    x = inputs.logits_normal(B, V, 4.0, dtype, seed=seed, device=dev)
    ctx = inputs.uniform_tokens((B, 1), V, seed=seed + 1, device=dev)
    want = oracle.bias_sample(inputs.as_oracle_array(x), V, ctx.cpu().numpy(), KEY, 0.25, 2.0, scheme, 0.7, 0xC4, step,
                              threads=8)

    def outs():
        return {"tokens": torch.full((B,), -1, dtype=torch.int32, device=dev),
                "max": torch.zeros(B, dtype=torch.float32, device=dev),
                "sumexp": torch.zeros(B, dtype=torch.float32, device=dev),
                "prob": torch.zeros(B, dtype=torch.float32, device=dev)}

    ref, got = outs(), outs()
    ws = torch.empty(sbw.sbw_sample_workspace_bytes(B, V), dtype=torch.uint8, device=dev)
    sbw.sbw_bias_sample(x, ctx, KEY, 0.25, 2.0, scheme, 0.7, 0xC4, step, ref["tokens"], ws,
                        out_max=ref["max"], out_sumexp=ref["sumexp"], out_prob=ref["prob"])
    sbw.sbw_bias_sample_noalloc(x, ctx, KEY, 0.25, 2.0, scheme, 0.7, 0xC4, step, got["tokens"],
                                out_max=got["max"], out_sumexp=got["sumexp"], out_prob=got["prob"])
    torch.cuda.synchronize()
    return ({k: v.cpu().numpy() for k, v in ref.items()}, {k: v.cpu().numpy() for k, v in got.items()}, want)


@pytest.mark.gpu
def test_noalloc_matches_workspace_entry_point_and_oracle_on_calls_in_a_row(oracle):
    dev = require_gpu()
    # first call: few rows, each split over many CTAs (uses partials and ticket counters); then the
    # same again; then more rows than any call before (parts of the array no call has cleared yet,
    # others holding stale partials and counters); then one row; then more rows again
    cases = [(8, 128256, torch.bfloat16, sbw.SCHEME_CONTEXT, 0, 11),
             (8, 128256, torch.bfloat16, sbw.SCHEME_CONTEXT, 1, 11),
             (300, 32000, torch.float32, sbw.SCHEME_SELFSALT, 2, 13),
             (1, 151936, torch.float32, sbw.SCHEME_CONTEXT, 3, 17),
             (700, 8192, torch.bfloat16, sbw.SCHEME_SELFSALT, 4, 19)]
    for B, V, dtype, scheme, step, seed in cases:
        ref, got, want = _both(dev, B, V, dtype, scheme, step, seed, oracle)
        assert np.array_equal(got["tokens"], ref["tokens"])
        assert np.array_equal(got["max"], ref["max"])
        assert np.max(np.abs(got["sumexp"] / ref["sumexp"] - 1.0)) <= REL
        assert np.max(np.abs(got["prob"] / ref["prob"] - 1.0)) <= REL
        assert got["tokens"].min() >= 0
        # and against the oracle: ids and maximum exactly, sum and probability to 1e-6
        assert np.array_equal(got["tokens"], want["tokens"])
        assert np.array_equal(got["max"].astype(np.float64), want["max"])
        assert np.max(np.abs(got["sumexp"].astype(np.float64) / want["sumexp"] - 1.0)) <= REL
        ok = want["prob"] >= np.finfo(np.float32).tiny
        assert np.max(np.abs(got["prob"].astype(np.float64)[ok] / want["prob"][ok] - 1.0)) <= REL


@pytest.mark.gpu
def test_noalloc_rejects_batches_beyond_its_capacity():
    dev = require_gpu()
    L = sbw.lib()
    B = binding.NOALLOC_MAX_ROWS + 1
    x = torch.zeros((B, 64), dtype=torch.float32, device=dev)
    ctx = torch.zeros((B, 1), dtype=torch.int32, device=dev)
    out = torch.full((B,), -5, dtype=torch.int32, device=dev)
    rc = L.sbw_bias_sample_noalloc(x.data_ptr(), 0, B, 64, 64, 0, ctx.data_ptr(), 1, KEY, 0.25, 2.0, 0,
                                   0.7, 1, 2, out.data_ptr(), None, None, None, None, None)
    assert rc == binding.SBW_ERR_TOO_LARGE
    torch.cuda.synchronize()
    assert int(out.max()) == -5                       # nothing was enqueued
    with pytest.raises(sbw.SbwError):
        sbw.sbw_bias_sample_noalloc(x, ctx, KEY, 0.25, 2.0, 0, 0.7, 1, 2, out)
    # the largest allowed batch works
    Bm = binding.NOALLOC_MAX_ROWS
    sbw.sbw_bias_sample_noalloc(x[:Bm], ctx[:Bm], KEY, 0.25, 2.0, 0, 0.7, 1, 2, out[:Bm])
    torch.cuda.synchronize()
    assert int(out[:Bm].min()) >= 0 and int(out[:Bm].max()) < 64
    assert isinstance(ctypes.c_int(rc).value, int)
