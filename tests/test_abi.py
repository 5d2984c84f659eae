"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
headers declare, and rejects bad arguments before touching the device."""
import ctypes
import re
from pathlib import Path

import pytest

import paper_2609_03844_b200 as sbw
from paper_2609_03844_b200 import binding

ROOT = Path(__file__).resolve().parent.parent


def _declared():
    names = set()
    for h in sorted((ROOT / "include").glob("*.h")):
        text = re.sub(r"/\*.*?\*/", "", h.read_text(), flags=re.S)
        names |= set(re.findall(r"\b(sbw_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_loads_and_exports_every_declared_symbol():
    L = sbw.lib()
    declared = _declared()
    assert {"sbw_bias_logits", "sbw_bias_sample", "sbw_detect", "sbw_version"} <= declared
    for name in declared:
        assert hasattr(L, name), f"{name} declared in include/ but not exported by libsbw.so"
    assert set(binding.EXPORTS) <= declared
    assert "sm_100a" in sbw.sbw_version()


def test_binding_has_the_same_names():
    for name in ("sbw_bias_logits", "sbw_bias_logits_host", "sbw_bias_sample", "sbw_detect",
                 "sbw_sample_workspace_bytes", "sbw_detect_workspace_bytes", "sbw_version"):
        assert callable(getattr(sbw, name))


def test_workspace_size_queries():
    assert sbw.sbw_sample_workspace_bytes(0, 128256) == 0
    a = sbw.sbw_sample_workspace_bytes(1, 128256)
    b = sbw.sbw_sample_workspace_bytes(1024, 128256)
    assert 0 < a < b and a % 256 == 0 and b % 256 == 0
    assert sbw.sbw_detect_workspace_bytes(0) == 0
    assert sbw.sbw_detect_workspace_bytes(100000) >= 8 * 100001
    assert sbw.sbw_bias_logits_host_staging_bytes(__import__("torch").bfloat16, 64, 128256, 1) >= \
        64 * 128256 * 2 + 64 * 4


def test_argument_validation_happens_on_the_host():
    """Every rejected call returns before any CUDA work, so this runs without a device."""
    L = sbw.lib()
    fake = ctypes.c_void_p(0x1000)          # never dereferenced on the host
    ok = dict(dtype=0, B=2, V=8, ld=8, off=0, W=1, key=1, gamma=0.25, delta=2.0, scheme=0)

    def bias(**kw):
        a = {**ok, **kw}
        return L.sbw_bias_logits(a.get("logits", fake), a["dtype"], a["B"], a["V"], a["ld"], a["off"],
                                 a.get("ctx", fake), a["W"], a["key"], a["gamma"], a["delta"],
                                 a["scheme"], None)

    assert bias(B=0) == binding.SBW_OK
    assert bias(B=0, logits=None, ctx=None) == binding.SBW_OK
    for bad in (dict(gamma=0.0), dict(gamma=1.0), dict(gamma=-0.1), dict(gamma=float("nan")),
                dict(V=0), dict(V=-3), dict(ld=7), dict(B=-1), dict(dtype=2), dict(scheme=5),
                dict(W=0), dict(W=9), dict(off=-1), dict(logits=None), dict(ctx=None),
                dict(delta=float("nan")), dict(delta=float("inf"))):
        assert bias(**bad) == binding.SBW_ERR_INVALID_ARG, bad
    assert bias(V=1 << 31, ld=1 << 31) == binding.SBW_ERR_UNSUPPORTED
    # delta = 0 is the paper's control: accepted, nothing to do
    assert bias(delta=0.0) == binding.SBW_OK

    def sample(**kw):
        a = {**ok, "tau": 0.7, "ws": fake, "ws_bytes": 1 << 20, **kw}
        return L.sbw_bias_sample(a.get("logits", fake), a["dtype"], a["B"], a["V"], a["ld"], a["off"],
                                 a.get("ctx", fake), a["W"], a["key"], a["gamma"], a["delta"],
                                 a["scheme"], a["tau"], 1, 2, a.get("out", fake), None, None, None,
                                 None, a["ws"], a["ws_bytes"], None)

    assert sample(B=0) == binding.SBW_OK
    for bad in (dict(tau=0.0), dict(tau=-1.0), dict(tau=float("nan")), dict(tau=1e-30),
                dict(gamma=1.5), dict(out=None), dict(logits=None), dict(ld=3)):
        assert sample(**bad) == binding.SBW_ERR_INVALID_ARG, bad
    assert sample(ws=None) == binding.SBW_ERR_WORKSPACE
    assert sample(ws_bytes=16) == binding.SBW_ERR_WORKSPACE
    assert sample(ws=ctypes.c_void_p(0x1008)) == binding.SBW_ERR_WORKSPACE   # not 256-aligned

    def noalloc(**kw):          # the entry without a workspace: same checks, then its capacity, all on the host
        a = {**ok, "tau": 0.7, **kw}
        return L.sbw_bias_sample_noalloc(a.get("logits", fake), a["dtype"], a["B"], a["V"], a["ld"], a["off"],
                                         a.get("ctx", fake), a["W"], a["key"], a["gamma"], a["delta"],
                                         a["scheme"], a["tau"], 1, 2, a.get("out", fake), None, None, None, None, None)

    assert noalloc(B=0) == binding.SBW_OK
    big = binding.NOALLOC_MAX_ROWS + 1
    assert noalloc(B=big) == binding.SBW_ERR_TOO_LARGE
    for bad in (dict(tau=0.0), dict(gamma=1.5), dict(out=None), dict(logits=None), dict(ld=3), dict(dtype=2),
                dict(delta=float("nan"))):
        assert noalloc(**bad) == binding.SBW_ERR_INVALID_ARG, bad
        assert noalloc(B=big, **bad) == binding.SBW_ERR_INVALID_ARG, bad      # the other fault is reported first

    def host(**kw):             # host-buffer entry: every check before the first copy is enqueued
        a = {**ok, "staging": ctypes.c_void_p(0x1000), "sb": 1 << 20, **kw}
        return L.sbw_bias_logits_host(a.get("logits", fake), a["dtype"], a["B"], a["V"], a["ld"], a["off"],
                                      a.get("ctx", fake), a["W"], a["key"], a["gamma"], a["delta"], a["scheme"],
                                      a["staging"], a["sb"], None)

    assert host(B=0) == binding.SBW_OK and host(delta=0.0) == binding.SBW_OK
    for bad in (dict(delta=float("nan")), dict(delta=float("inf")), dict(gamma=0.0), dict(logits=None), dict(ctx=None)):
        assert host(**bad) == binding.SBW_ERR_INVALID_ARG, bad
    assert host(off=(1 << 32) - 4) == binding.SBW_ERR_UNSUPPORTED
    assert host(staging=None) == binding.SBW_ERR_WORKSPACE and host(sb=8) == binding.SBW_ERR_WORKSPACE

    def shard(**kw):            # a shard summary holds the global id in 31 bits
        a = {**ok, "tau": 0.7, **kw}
        return L.sbw_bias_sample_shard(fake, a["dtype"], a["B"], a["V"], a["ld"], a["off"], 0, fake, a["W"], a["key"],
                                       a["gamma"], a["delta"], a["scheme"], a["tau"], 1, 2, a.get("summary", fake), fake,
                                       fake, 1 << 20, None)

    assert shard(B=0) == binding.SBW_OK
    assert shard(off=(1 << 31) - 4) == binding.SBW_ERR_UNSUPPORTED
    assert shard(summary=None) == binding.SBW_ERR_INVALID_ARG

    def detect(**kw):
        a = dict(N=4, total=40, W=1, gamma=0.25, scheme=0, ws=fake, ws_bytes=1 << 20, off=None)
        a.update(kw)
        return L.sbw_detect(a.get("tokens", fake), a.get("lengths", fake), a["off"], a["N"], a["total"],
                            a["W"], 1, a["gamma"], a["scheme"], a.get("counts", fake), None,
                            a.get("z", fake), a["ws"], a["ws_bytes"], None)

    assert detect(N=0) == binding.SBW_OK
    for bad in (dict(gamma=0.0), dict(N=-1), dict(total=-5), dict(W=0), dict(scheme=2),
                dict(lengths=None), dict(counts=None), dict(z=None), dict(tokens=None)):
        assert detect(**bad) == binding.SBW_ERR_INVALID_ARG, bad
    assert detect(ws=None, ws_bytes=0) == binding.SBW_ERR_WORKSPACE
    assert detect(ws_bytes=8) == binding.SBW_ERR_WORKSPACE
    assert L.sbw_last_cuda_error() == 0


def test_argument_validation_of_the_widened_entry_points():
    """Same for the calls added after the first three: bad arguments come back before any CUDA work."""
    L = sbw.lib()
    fake = ctypes.c_void_p(0x1000)
    INV, UNS, WSP, OK = (binding.SBW_ERR_INVALID_ARG, binding.SBW_ERR_UNSUPPORTED, binding.SBW_ERR_WORKSPACE,
                         binding.SBW_OK)

    def topk(**kw):
        a = dict(logits=fake, dtype=0, B=2, V=8, ld=8, off=0, ctx=fake, W=1, gamma=0.25, delta=2.0, scheme=1, k=3)
        a.update(kw)
        return L.sbw_bias_logits_topk(a["logits"], a["dtype"], a["B"], a["V"], a["ld"], a["off"], a["ctx"], a["W"], 1,
                                      a["gamma"], a["delta"], a["scheme"], a["k"], None)

    assert topk(B=0) == OK and topk(delta=0.0) == OK
    for bad in (dict(k=0), dict(k=-2), dict(gamma=1.0), dict(V=0), dict(ld=4), dict(logits=None), dict(ctx=None),
                dict(delta=float("nan")), dict(W=9)):
        assert topk(**bad) == INV, bad

    def filtered(**kw):
        a = dict(logits=fake, dtype=1, B=2, V=64, ld=64, off=0, ctx=fake, W=1, gamma=0.25, delta=2.0, scheme=0,
                 tau=0.7, k=0, p=0.8, out=fake, ws=fake, ws_bytes=1 << 20)
        a.update(kw)
        return L.sbw_bias_sample_filtered(a["logits"], a["dtype"], a["B"], a["V"], a["ld"], a["off"], a["ctx"],
                                          a["W"], 1, a["gamma"], a["delta"], a["scheme"], a["tau"], a["k"], a["p"],
                                          1, 2, a["out"], None, a["ws"], a["ws_bytes"], None)

    assert filtered(B=0) == OK
    for bad in (dict(p=0.0), dict(p=-1.0), dict(p=float("nan")), dict(k=-1), dict(tau=0.0), dict(gamma=0.0),
                dict(V=0), dict(ld=8), dict(out=None), dict(logits=None), dict(ctx=None), dict(off=-1)):
        assert filtered(**bad) == INV, bad
    assert filtered(V=(1 << 21) + 8, ld=(1 << 21) + 8) == UNS
    assert filtered(ws=None) == WSP and filtered(ws_bytes=64) == WSP
    assert L.sbw_sample_filtered_workspace_bytes(1, 2, 64) >= 2 * 64 * 2
    assert L.sbw_sample_filtered_workspace_bytes(7, 2, 64) == 0

    def unique(**kw):
        a = dict(tokens=fake, lengths=fake, off=None, N=4, total=40, maxlen=10, W=1, gamma=0.25, scheme=0,
                 counts=fake, z=fake, ws=fake, ws_bytes=1 << 20)
        a.update(kw)
        return L.sbw_detect_unique(a["tokens"], a["lengths"], a["off"], a["N"], a["total"], a["maxlen"], a["W"], 1,
                                   a["gamma"], a["scheme"], a["counts"], None, a["z"], a["ws"], a["ws_bytes"], None)

    assert unique(N=0) == OK
    for bad in (dict(gamma=1.0), dict(N=-1), dict(total=-1), dict(maxlen=-1), dict(W=0), dict(scheme=3),
                dict(lengths=None), dict(counts=None), dict(z=None), dict(tokens=None)):
        assert unique(**bad) == INV, bad
    assert unique(ws=None) == WSP and unique(ws_bytes=8) == WSP
    assert L.sbw_detect_unique_workspace_bytes(4, 40, 5000) >= 16 * 40

    def prefix(**kw):
        a = dict(bits=fake, lengths=fake, off=fake, keep=fake, N=4, total=40, W=1, gamma=0.25, counts=fake, z=fake)
        a.update(kw)
        return L.sbw_prefix_z(a["bits"], a["lengths"], a["off"], a["keep"], a["N"], a["total"], a["W"], a["gamma"],
                              a["counts"], None, a["z"], None)

    assert prefix(N=0) == OK
    for bad in (dict(gamma=0.0), dict(W=9), dict(N=-1), dict(bits=None), dict(off=None), dict(keep=None),
                dict(counts=None), dict(z=None)):
        assert prefix(**bad) == INV, bad

    def roc(**kw):
        a = dict(z=fake, labels=fake, n=10, auc=fake, ws=fake, ws_bytes=1 << 20)
        a.update(kw)
        return L.sbw_roc_auc(a["z"], a["labels"], a["n"], a["auc"], None, a["ws"], a["ws_bytes"], None)

    for bad in (dict(n=-1), dict(auc=None), dict(z=None), dict(labels=None)):
        assert roc(**bad) == INV, bad
    assert roc(n=(1 << 31) + 1, ws_bytes=1 << 40) == UNS
    assert roc(ws=None) == WSP and roc(ws_bytes=16) == WSP
    assert L.sbw_roc_auc_batched(fake, fake, fake, 0, fake, None, None) == OK
    assert L.sbw_roc_auc_batched(fake, fake, None, 3, fake, None, None) == INV
    assert L.sbw_roc_auc_batched(fake, fake, fake, -1, fake, None, None) == INV
    assert L.sbw_last_cuda_error() == 0


def test_python_binding_type_checks():
    import torch

    with pytest.raises(ValueError):
        sbw.sbw_bias_logits(torch.zeros(2, 8), torch.zeros(2, 1, dtype=torch.int32), 1, 0.25, 2.0, 0)
