"""Pins for the oracle's top-k / top-p sampling (Appendix F samples with top_p = 0.8).  The kept
set is checked against an fp64 softmax with cumulative sums in numpy, torch.topk, closed forms,
and the sampled ids against the truncated, renormalised distribution by chi-square."""
import numpy as np
import pytest
import torch
from scipy import stats

import oracle
from paper_2609_03844_b200 import inputs

KEY = 0x5EED


def _biased(x, V, ctx, gamma, delta, scheme):
    return oracle.bias_logits(x, V, ctx, KEY, gamma, delta, scheme)


def _bf16_to_f32(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32)


def test_weight_is_two_to_the_scaled_difference():
    c = np.float32(1.4426950408889634 / 0.7)
    rng = np.random.default_rng(0)
    m = np.float32(7.25)
    for l in (m - rng.random(2000).astype(np.float32) * np.float32(21.0)):
        w = oracle.nucleus_weight(float(l), float(m), False, float(c))
        y = float(np.float32(np.float32(l - m) * c))
        ref = 2.0 ** (y + 40)
        if y >= -41:
            assert abs(w - ref) <= 2e-7 * ref + 1
        else:
            assert w == 0
    assert oracle.nucleus_weight(3.0, 3.0, True, float(c)) == 1 << 40
    assert oracle.nucleus_weight(0.0, 0.0, False, float(c)) == 1 << 40      # -0 against +0: y = 0
    assert oracle.nucleus_weight(float("-inf"), 1.0, False, float(c)) == 0
    assert oracle.nucleus_weight(float("nan"), 1.0, False, float(c)) == 0
    # monotone in the logit, so the order of the weights is the order of the candidates
    ls = np.sort(rng.normal(0, 4, 3000).astype(np.float32))
    ws = [oracle.nucleus_weight(float(l), float(ls[-1]), False, float(c)) for l in ls]
    assert all(a <= b for a, b in zip(ws, ws[1:]))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("top_p", [0.8, 0.5, 0.95, 0.999])
def test_nucleus_matches_fp64_softmax(dtype, top_p):
    B, V, tau = 6, 5000, 0.7
    x = inputs.as_oracle_array(inputs.logits_normal(B, V, 2.0, dtype, seed=3))
    ctx = inputs.uniform_tokens((B, 1), V, seed=4).numpy()
    got = oracle.bias_sample_filtered(x, V, ctx, KEY, 0.25, 2.0, 1, tau, 0, top_p, 7, 0, want_mask=True)
    lb = _biased(x, V, ctx, 0.25, 2.0, 1)
    lb = _bf16_to_f32(lb) if lb.dtype == np.uint16 else lb
    for b in range(B):
        z = lb[b].astype(np.float64) / tau
        p = np.exp(z - z.max())
        p /= p.sum()
        order = np.lexsort((np.arange(V), -lb[b].astype(np.float64)))       # value desc, column asc
        before = np.concatenate([[0.0], np.cumsum(p[order])[:-1]])
        keep = before < top_p
        n = int(keep.sum())
        # the cut may move where the cumulative mass is within the weights' rounding of top_p
        slack = np.abs(before - top_p) < 1e-5
        assert abs(int(got["kept"][b]) - n) <= int(slack.sum())
        want = np.zeros(V, dtype=np.uint8)
        want[order[:got["kept"][b]]] = 1
        assert np.array_equal(got["mask"][b], want)                          # always a prefix of the order
        assert got["mask"][b][got["tokens"][b]] == 1


def test_top_k_alone_is_torch_topk():
    B, V, k = 4, 3000, 50
    x = inputs.logits_normal(B, V, 4.0, torch.float32, seed=9)
    ctx = inputs.uniform_tokens((B, 1), V, seed=10).numpy()
    got = oracle.bias_sample_filtered(x.numpy(), V, ctx, KEY, 0.5, 2.0, 0, 1.0, k, 1.0, 1, 1, want_mask=True)
    lb = torch.from_numpy(_biased(x.numpy(), V, ctx, 0.5, 2.0, 0))
    idx = torch.topk(lb, k, dim=1).indices.numpy()
    for b in range(B):
        assert set(np.flatnonzero(got["mask"][b])) == set(idx[b]) and got["kept"][b] == k


def test_filters_off_is_the_plain_sampler():
    B, V = 5, 4000
    x = inputs.as_oracle_array(inputs.logits_normal(B, V, 4.0, torch.bfloat16, seed=12))
    ctx = inputs.uniform_tokens((B, 1), V, seed=13).numpy()
    for step in range(4):
        a = oracle.bias_sample_filtered(x, V, ctx, KEY, 0.25, 2.0, 1, 0.7, 0, 1.0, 99, step)
        b = oracle.bias_sample(x, V, ctx, KEY, 0.25, 2.0, 1, 0.7, 99, step)
        assert np.array_equal(a["tokens"], b["tokens"]) and (a["kept"] == V).all()
        a = oracle.bias_sample_filtered(x, V, ctx, KEY, 0.25, 2.0, 1, 0.7, V + 5, 1.5, 99, step)
        assert np.array_equal(a["tokens"], b["tokens"])


def test_closed_forms():
    V = 10
    flat = np.zeros((1, V), dtype=np.float32)
    ctx = [[3]]
    # equal logits and delta = 0: equal weights, so top_p keeps ceil(top_p V) lowest columns
    for top_p, n in ((0.5, 5), (0.31, 4), (0.05, 1), (1e-12, 1), (0.9999, 10)):
        r = oracle.bias_sample_filtered(flat, V, ctx, KEY, 0.5, 0.0, 0, 1.0, 0, top_p, 1, 0, want_mask=True)
        assert r["kept"][0] == n and r["mask"][0].tolist() == [1] * n + [0] * (V - n)
    # one dominant logit: any top_p below its probability is greedy decoding
    x = np.full((1, V), -5.0, dtype=np.float32)
    x[0, 6] = 9.0
    for step in range(5):
        r = oracle.bias_sample_filtered(x, V, ctx, KEY, 0.5, 0.0, 0, 1.0, 0, 0.99, 5, step)
        assert r["tokens"][0] == 6 and r["kept"][0] == 1
    # top-k then top-p: the nucleus is taken inside the top-k set (renormalised)
    y = np.array([[4.0, 3.0, 2.0, 1.0, 0.0, -1.0]], dtype=np.float32)
    p = np.exp(y[0, :3].astype(np.float64))
    p /= p.sum()                                             # softmax over the top 3 only
    r = oracle.bias_sample_filtered(y, 6, ctx, KEY, 0.5, 0.0, 0, 1.0, 3, float(p[0] + 0.01), 5, 0)
    assert r["kept"][0] == 2
    r = oracle.bias_sample_filtered(y, 6, ctx, KEY, 0.5, 0.0, 0, 1.0, 3, float(p[0] - 0.01), 5, 0)
    assert r["kept"][0] == 1
    # ties at the cut go to the lowest columns; top_k = 1 is the arg max with ties to the lowest id
    t = np.array([[1.0, 2.0, 2.0, 2.0, 0.0]], dtype=np.float32)
    r = oracle.bias_sample_filtered(t, 5, ctx, KEY, 0.5, 0.0, 0, 1.0, 2, 1.0, 5, 0, want_mask=True)
    assert r["mask"][0].tolist() == [0, 1, 1, 0, 0]
    r = oracle.bias_sample_filtered(t, 5, ctx, KEY, 0.5, 0.0, 0, 1.0, 1, 1.0, 5, 0)
    assert r["tokens"][0] == 1


def test_sampled_ids_follow_the_truncated_distribution():
    V, tau, top_p, steps = 40, 0.7, 0.8, 6000
    x = inputs.logits_normal(1, V, 1.0, torch.float32, seed=21).numpy()
    ctx = [[5]]
    lb = _biased(x, V, ctx, 0.25, 1.0, 0)[0].astype(np.float64)
    r = oracle.bias_sample_filtered(x, V, ctx, KEY, 0.25, 1.0, 0, tau, 0, top_p, 3, 0, want_mask=True)
    mask = r["mask"][0].astype(bool)
    p = np.exp((lb - lb.max()) / tau) * mask
    p /= p.sum()
    xs = np.repeat(x, steps, axis=0)                          # same logits in every row: rows differ by RNG
    ids = oracle.bias_sample_filtered(xs, V, np.repeat(ctx, steps, axis=0), KEY, 0.25, 1.0, 0, tau, 0, top_p,
                                      3, 0, threads=4)["tokens"]
    assert mask[ids].all()
    obs = np.bincount(ids, minlength=V)[mask]
    exp = p[mask] * steps
    assert exp.min() > 5
    assert stats.chisquare(obs, exp).pvalue > 1e-3
