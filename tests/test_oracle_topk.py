"""Pins for the oracle's top-k candidate restriction (the paper's SBW-ss scheme: self-salt on the
top-40 candidates): the selection against torch.topk and brute force, the bias against the
full-vocabulary oracle restricted to the chosen columns."""
import numpy as np
import pytest
import torch

from paper_2609_03844_b200 import inputs

KEY = 0x5EED


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("k", [1, 40, 100])
def test_selection_matches_torch_topk_values(oracle, dtype, k):
    B, V = 6, 5000
    x = inputs.logits_normal(B, V, 4.0, dtype, seed=50 + k)
    arr = inputs.as_oracle_array(x)
    ctx = inputs.uniform_tokens((B, 1), V, seed=51).numpy()
    _, sel = oracle.bias_logits_topk(arr, V, ctx, KEY, 0.25, 2.0, oracle.SCHEME_SELFSALT, k)
    want_vals = torch.topk(x.float(), k, dim=1).values.numpy()
    got_vals = np.take_along_axis(x.float().numpy(), sel.astype(np.int64), axis=1)
    assert np.array_equal(got_vals, want_vals)                    # same multiset, rank order
    for b in range(B):
        assert len(set(sel[b])) == k
        # ties go to the lowest columns: within equal values the chosen columns ascend, and no
        # unchosen column with the k-th value precedes a chosen one
        kth = got_vals[b, -1]
        same = np.flatnonzero(x[b].float().numpy() == kth)
        chosen_same = sorted(c for c in sel[b] if x[b, c].float() == kth)
        assert chosen_same == list(same[:len(chosen_same)])


def test_selection_brute_force_with_ties_zeros_and_infinities(oracle):
    vals = np.array([0.0, -0.0, 1.5, 1.5, -np.inf, np.inf, 1.5, 0.0, -2.0, np.inf, -0.0, 1.5],
                    dtype=np.float32)
    x = vals.reshape(1, -1)
    ctx = np.array([[3]], dtype=np.int32)
    # total order: +inf (cols 5, 9), 1.5 (2, 3, 6, 11), +0.0 (0, 7), -0.0 (1, 10), -2.0 (8), -inf (4)
    full = [5, 9, 2, 3, 6, 11, 0, 7, 1, 10, 8, 4]
    for k in range(1, 13):
        _, sel = oracle.bias_logits_topk(x, 12, ctx, KEY, 0.5, 1.0, oracle.SCHEME_SELFSALT, k)
        assert list(sel[0]) == full[:k]
    _, sel = oracle.bias_logits_topk(x, 12, ctx, KEY, 0.5, 1.0, oracle.SCHEME_SELFSALT, 40)
    assert list(sel[0]) == full                                   # k > V: every column


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("scheme_name", ["context", "selfsalt"])
def test_bias_equals_full_vocabulary_bias_on_the_chosen_columns(oracle, dtype, scheme_name):
    scheme = oracle.SCHEME_SELFSALT if scheme_name == "selfsalt" else oracle.SCHEME_CONTEXT
    B, V, ld, off, k = 4, 3001, 3008, 11, 40
    x = inputs.logits_normal(B, V, 4.0, dtype, seed=60, ld=ld)
    arr = inputs.as_oracle_array(x)
    ctx = inputs.uniform_tokens((B, 4), 151936, seed=61).numpy()
    got, sel = oracle.bias_logits_topk(arr, V, ctx, KEY, 0.25, 2.0, scheme, k, vocab_offset=off)
    full = oracle.bias_logits(arr, V, ctx, KEY, 0.25, 2.0, scheme, vocab_offset=off)
    want = arr.copy()
    for b in range(B):
        want[b, sel[b]] = full[b, sel[b]]
    assert got.tobytes() == want.tobytes()
    changed = (got != arr).sum(axis=1)
    assert np.all(changed <= k) and changed.sum() > 0
    # k >= V is the full-vocabulary scheme
    allv, _ = oracle.bias_logits_topk(arr, V, ctx, KEY, 0.25, 2.0, scheme, V + 5, vocab_offset=off)
    assert allv.tobytes() == full.tobytes()
