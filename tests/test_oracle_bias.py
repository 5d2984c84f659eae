"""Pins for the oracle's bias step (Eq. 2): IEEE adds against numpy / torch, bit-identity of
non-green elements, and the whole in-place step against mask-then-add written with library ops."""
import numpy as np
import pytest
import torch

from paper_2609_03844_b200 import inputs

KEY = 0x5EED


def test_f32_add_matches_numpy(oracle):
    rng = np.random.default_rng(20)
    xs = np.concatenate([rng.normal(0, 4, 5000).astype(np.float32),
                         np.array([0.0, -0.0, np.inf, -np.inf, 1e-45, -1e-45, 3.4e38, -3.4e38,
                                   16777216.0, 1e-30], dtype=np.float32)])
    for delta in (2.0, 0.5, 0.1, -1.25, 4.0, 1e-8):
        d32 = np.float32(delta)
        for x in xs:
            got = np.float32(oracle.lib().sbw_oracle_bias_elem_f32(float(x), float(d32), 1))
            with np.errstate(over="ignore"):
                want = np.float32(x + d32)
            assert got.tobytes() == want.tobytes() or (np.isnan(got) and np.isnan(want))
            same = np.float32(oracle.lib().sbw_oracle_bias_elem_f32(float(x), float(d32), 0))
            assert same.tobytes() == np.float32(x).tobytes()


@pytest.mark.parametrize("delta", [0.5, 1.0, 2.0, 4.0, 0.3, -1.5, 0.0])
def test_bf16_add_matches_torch_on_every_bit_pattern(oracle, delta):
    """All 65536 bf16 inputs: green elements equal torch's bfloat16 addition of delta rounded to
    bf16; non-green elements keep their bits."""
    bits = np.arange(65536, dtype=np.uint16)
    logits = bits.reshape(1, -1).copy()
    # one call with every element green (gamma ~ 1) and one with none green is not available
    # through the mask, so use the element function directly
    L = oracle.lib()
    got = np.array([L.sbw_oracle_bias_elem_bf16(int(b), delta, 1) for b in bits], dtype=np.uint16)
    t = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)
    d = torch.tensor(delta, dtype=torch.float32).to(torch.bfloat16)
    want = (t + d).view(torch.int16).numpy().view(np.uint16)
    if float(d) == 0.0:
        want = bits        # the paper's delta = 0 control: no add at all, -0.0 stays -0.0
    nan = torch.isnan(t).numpy()
    assert np.array_equal(got[~nan], want[~nan])
    g32 = torch.from_numpy(got.view(np.int16).copy()).view(torch.bfloat16)
    assert bool(torch.isnan(g32[torch.from_numpy(nan)]).all())
    same = np.array([L.sbw_oracle_bias_elem_bf16(int(b), delta, 0) for b in bits], dtype=np.uint16)
    assert np.array_equal(same, bits)
    del logits


def test_bf16_narrowing_matches_torch(oracle):
    rng = np.random.default_rng(21)
    xs = np.concatenate([rng.normal(0, 10, 20000), rng.normal(0, 1e-3, 2000),
                         [0.0, -0.0, 1.00390625, 1.01171875, 3.3895313892515355e38, 3.4e38,
                          np.inf, -np.inf, 1e-40, 9.18e-41]]).astype(np.float32)
    want = torch.from_numpy(xs).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.lib().sbw_oracle_f32_to_bf16(float(x)) for x in xs], dtype=np.uint16)
    assert np.array_equal(got, want)
    back = np.array([oracle.lib().sbw_oracle_bf16_to_f32(int(h)) for h in got], dtype=np.float32)
    assert np.array_equal(back, torch.from_numpy(xs).to(torch.bfloat16).float().numpy())


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("scheme_name", ["context", "selfsalt"])
def test_step_equals_mask_then_library_add(oracle, dtype, scheme_name):
    """Eq. 2 for a whole step = where(mask, l + delta, l) with torch's own add; padding columns
    (ld > V) untouched; delta = 0 leaves every bit alone (the paper's delta = 0 control)."""
    scheme = oracle.SCHEME_SELFSALT if scheme_name == "selfsalt" else oracle.SCHEME_CONTEXT
    B, V, ld, off = 5, 1003, 1016, 17
    x = inputs.logits_normal(B, V, 4.0, dtype, seed=22, ld=ld)
    x[0, 0] = -0.0
    x[1, 1] = float("-inf")
    ctx = inputs.uniform_tokens((B, 1), 50000, seed=23).numpy()
    gamma, delta = 0.25, 2.0
    mask = oracle.green_mask(B, V, ctx, KEY, gamma, scheme, vocab_offset=off).astype(bool)
    arr = inputs.as_oracle_array(x)
    got = oracle.bias_logits(arr, V, ctx, KEY, gamma, delta, scheme, vocab_offset=off)
    want_t = x.clone()
    body = want_t[:, :V]
    body[torch.from_numpy(mask)] = (body + torch.tensor(delta).to(dtype))[torch.from_numpy(mask)]
    want = inputs.as_oracle_array(want_t)
    assert got.tobytes() == want.tobytes()
    assert np.array_equal(got[:, V:], arr[:, V:])
    assert 0.15 < mask.mean() < 0.35
    zero = oracle.bias_logits(arr, V, ctx, KEY, gamma, 0.0, scheme, vocab_offset=off)
    assert zero.tobytes() == arr.tobytes()
    # rows split over threads give the same bytes
    mt = oracle.bias_logits(arr, V, ctx, KEY, gamma, delta, scheme, vocab_offset=off, threads=3)
    assert mt.tobytes() == got.tobytes()
