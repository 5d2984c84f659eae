"""The bounds-flag build of the library (-DSBW_DEBUG): every global access of the bias, sample and
detect kernels is preceded by a check of its indices against the call's sizes; a failed check is
recorded in a device flag and the access skipped (nothing traps).  This stands in for a memory
checker, which cannot be run on the machines this library is tested on.  The shapes are the
awkward small ones -- one to nine columns, rows that are not 16-byte aligned, padded strides,
sequences shorter than the context -- and every result is also compared with the oracle."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2609_03844_b200 import build as sbw_build, inputs
from gpu_util import KEY, assert_same_bits, host_bits, require_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dbg():
    require_gpu()
    path = sbw_build.build(debug=True)              # compiled here if missing or older than the sources
    L = ctypes.CDLL(str(path))
    c = ctypes
    i64, u64, i32, vp, sz = c.c_int64, c.c_uint64, c.c_int, c.c_void_p, c.c_size_t
    L.sbw_bias_logits.restype = i32
    L.sbw_bias_logits.argtypes = [vp, i32, i64, i64, i64, i64, vp, i32, u64, c.c_double, c.c_float, i32, vp]
    L.sbw_sample_workspace_bytes.restype = sz
    L.sbw_sample_workspace_bytes.argtypes = [i64, i64]
    L.sbw_bias_sample.restype = i32
    L.sbw_bias_sample.argtypes = [vp, i32, i64, i64, i64, i64, vp, i32, u64, c.c_double, c.c_float, i32, c.c_float,
                                  u64, u64, vp, vp, vp, vp, vp, vp, sz, vp]
    L.sbw_detect_workspace_bytes.restype = sz
    L.sbw_detect_workspace_bytes.argtypes = [i64]
    L.sbw_detect.restype = i32
    L.sbw_detect.argtypes = [vp, vp, vp, i64, i64, i32, u64, c.c_double, i32, vp, vp, vp, vp, sz, vp]
    L.sbw_debug_flags.restype = i32
    L.sbw_debug_flags.argtypes = [vp, i32]
    L.sbw_debug_selftest.restype = i32
    L.sbw_debug_selftest.argtypes = [vp]
    return L


def _flags(L, clear=True):
    out = (ctypes.c_uint * 4)()
    assert L.sbw_debug_flags(out, 1 if clear else 0) == 0
    return list(out)


def test_the_flag_records_a_failed_check_without_faulting(dbg):
    _flags(dbg)
    assert dbg.sbw_debug_selftest(None) == 0
    mask, failures, passed, _ = _flags(dbg)
    assert mask == 1 << 31 and failures == 1 and passed == 1
    assert _flags(dbg) == [0, 0, 0, 0]                       # cleared
    x = torch.zeros(8, device="cuda")                        # the context is still usable
    assert float((x + 1).sum()) == 8.0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("scheme", [0, 1])
def test_bias_and_sample_on_awkward_shapes_pass_every_check(dbg, oracle, dtype, scheme):
    dev = torch.device("cuda:0")
    code = 0 if dtype == torch.float32 else 1
    stream = torch.cuda.current_stream().cuda_stream
    _flags(dbg)
    for B, V, ld, skew in ((1, 1, 1, 0), (2, 3, 3, 0), (3, 7, 7, 0), (2, 8, 8, 0), (3, 9, 16, 0), (2, 33, 40, 1),
                           (4, 1000, 1003, 0), (5, 4099, 4104, 3), (2, 32000, 32000, 0)):
        full = inputs.logits_normal(B, V, 4.0, dtype, seed=V + B, ld=ld + skew)
        rows = full[:, skew:skew + ld]                        # skew: rows that do not start on 16-byte boundaries
        ctx = inputs.uniform_tokens((B, 2), max(V, 2), seed=V)
        host = host_bits(rows.contiguous())
        dfull, dctx = full.to(dev), ctx.to(dev)
        drows = dfull[:, skew:skew + ld]
        # sample first (read only), then bias in place
        ids = torch.empty(B, dtype=torch.int32, device=dev)
        Z = torch.empty(B, dtype=torch.float32, device=dev)
        ws = torch.empty(max(dbg.sbw_sample_workspace_bytes(B, V), 256), dtype=torch.uint8, device=dev)
        rc = dbg.sbw_bias_sample(drows.data_ptr(), code, B, V, drows.stride(0), 5, dctx.data_ptr(), 2, KEY, 0.25, 2.0,
                                 scheme, 0.7, 3, 4, ids.data_ptr(), None, Z.data_ptr(), None, None, ws.data_ptr(),
                                 ws.numel(), stream)
        assert rc == 0
        rc = dbg.sbw_bias_logits(drows.data_ptr(), code, B, V, drows.stride(0), 5, dctx.data_ptr(), 2, KEY, 0.25, 2.0,
                                 scheme, stream)
        assert rc == 0
        torch.cuda.synchronize()
        want = oracle.bias_logits(host, V, ctx.numpy(), KEY, 0.25, 2.0, scheme, vocab_offset=5)
        assert_same_bits(host_bits(drows.contiguous()), want)
        ws_o = oracle.bias_sample(host, V, ctx.numpy(), KEY, 0.25, 2.0, scheme, 0.7, 3, 4, vocab_offset=5)
        assert np.array_equal(ids.cpu().numpy(), ws_o["tokens"])
        assert np.max(np.abs(Z.cpu().numpy() / ws_o["sumexp"] - 1)) <= 1e-6
    mask, failures, passed, _ = _flags(dbg)
    assert mask == 0 and failures == 0 and passed > 0


@pytest.mark.parametrize("scheme", [0, 1])
@pytest.mark.parametrize("width", [1, 4, 7])
def test_detect_on_awkward_sequences_passes_every_check(dbg, oracle, scheme, width):
    dev = torch.device("cuda:0")
    stream = torch.cuda.current_stream().cuda_stream
    _flags(dbg)
    for N, lmin, lmax in ((1, 0, 0), (3, 0, 9), (40, 0, 300), (2000, 0, 200), (5, 1000, 5000)):
        tokens, lengths = inputs.null_token_streams(N, lmin, lmax, 5000, seed=N + width)
        if tokens.numel() == 0:
            tokens = torch.zeros(1, dtype=torch.int32)       # a valid pointer; total_tokens stays 0
            total = 0
        else:
            total = tokens.numel()
        dtok, dlen = tokens.to(dev), lengths.to(dev)
        counts = torch.full((N,), -7, dtype=torch.int32, device=dev)
        T = torch.full((N,), -7, dtype=torch.int32, device=dev)
        z = torch.zeros(N, dtype=torch.float64, device=dev)
        ws = torch.empty(max(dbg.sbw_detect_workspace_bytes(N), 256), dtype=torch.uint8, device=dev)
        rc = dbg.sbw_detect(dtok.data_ptr(), dlen.data_ptr(), None, N, total, width, KEY, 0.25, scheme, counts.data_ptr(),
                            T.data_ptr(), z.data_ptr(), ws.data_ptr(), ws.numel(), stream)
        assert rc == 0
        torch.cuda.synchronize()
        oc, oT, oz = oracle.detect(tokens.numpy()[:total], lengths.numpy(), KEY, 0.25, scheme, ctx_width=width)
        assert np.array_equal(counts.cpu().numpy(), oc) and np.array_equal(T.cpu().numpy(), oT)
        assert np.max(np.abs(z.cpu().numpy() - oz), initial=0.0) <= 1e-9
    mask, failures, passed, _ = _flags(dbg)
    assert mask == 0 and failures == 0 and passed > 0
