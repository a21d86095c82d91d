"""Parity of hilore_plan_apply with the CPU oracle: psi / action / recompute / retained bytes bit-exact
on the same exposure bits; the batched capture / encode / recover phases touch exactly the units the
gates select (H bundles stay byte-identical, R units' buffers are never written)."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_2609_33570_b200 import api, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu
R, H, L = api.ACT_R, api.ACT_H, api.ACT_L


def decide(table_dev, table_host, U, exposure, kappa, ebar, tau_lo, tau_hi, avail, action_in=None):
    act = G.Guarded(U)
    if action_in is not None:
        act.view.copy_(G.dev(np.asarray(action_in, np.uint8)))
    psi, rec, ret = G.Guarded(U * 4), G.Guarded(U), G.Guarded(U * 8)
    api.hilore_plan_apply(table_dev, table_host, U, api.PHASE_DECIDE,
                          None if exposure is None else G.dev(exposure),
                          None if exposure is None else G.dev(kappa), None if exposure is None else G.dev(ebar),
                          tau_lo, tau_hi, G.dev(np.asarray(avail, np.uint8)), act.ptr(), psi.ptr(), rec.ptr(), ret.ptr())
    return (act.numpy(np.uint8, (U,)), psi.numpy(np.float32, (U,)), rec.numpy(np.uint8, (U,)),
            ret.numpy(np.uint64, (U,)))


def shapes_table(shapes, fmts):
    units = [dict(rows=r, cols=c, fmt=f, block=0 if f == api.FMT_E4M3FN_RAW else 64) for (r, c), f in zip(shapes, fmts)]
    return api.make_unit_table(units), units


def test_decide_availability_table_exhaustive():
    combos = list(itertools.product((R, H, L), repeat=2))
    (dev, host), units = shapes_table([(128, 256)] * 9, [api.FMT_E4M3FN_BLK] * 9)
    want = [w for w, _ in combos]
    avail = [q for _, q in combos]
    a, _, rec, ret = decide(dev, host, 9, None, None, None, 0, 0, avail, action_in=want)
    oa, _, orec, oret = oracle.plan(None, None, None, 0, 0, avail, [128] * 9, [256] * 9, [1] * 9, [64] * 9, action_in=want)
    assert np.array_equal(a, oa) and np.array_equal(rec, orec) and np.array_equal(ret, oret)
    allowed = {H: {H, L, R}, L: {L, R}, R: {R}}
    assert a.tolist() == [w if w in allowed[q] else R for w, q in combos]


def test_decide_thresholds_config3_quantiles():
    """U = 84 (28 layers x 3 units), thresholds at midpoints between order statistics: 42 L / 25 H / 17 R."""
    rng = np.random.default_rng(0)
    U = 84
    shapes = [(16384, d) for _ in range(28) for d in (3584, 3584, 18944)]
    fmts = [api.FMT_E4M3FN_BLK, api.FMT_E4M3FN_RAW, api.FMT_INT8_BLK] * 28
    (dev, host), units = shapes_table(shapes, fmts)
    exposure = (rng.random(U, dtype=np.float32) + np.float32(0.1))
    kappa = rng.uniform(0.5, 2.0, U).astype(np.float32)
    ebar = np.full(U, 0.0266, np.float32)
    psi_ref = (kappa * exposure).astype(np.float32) * ebar
    srt = np.sort(psi_ref)
    tau_lo = float((srt[41] + srt[42]) / 2)
    tau_hi = float((srt[U - 26] + srt[U - 25]) / 2)
    for avail in ([H] * U, [(H, L, R, H)[i % 4] for i in range(U)]):
        a, psi, rec, ret = decide(dev, host, U, exposure, kappa, ebar, tau_lo, tau_hi, avail)
        oa, opsi, orec, oret = oracle.plan(exposure, kappa, ebar, tau_lo, tau_hi, avail, [s[0] for s in shapes],
                                           [s[1] for s in shapes], fmts, [u["block"] for u in units])
        assert np.array_equal(psi.view(np.uint32), opsi.view(np.uint32))
        assert np.array_equal(a, oa) and np.array_equal(rec, orec) and np.array_equal(ret, oret)
    a, *_ = decide(dev, host, U, exposure, kappa, ebar, tau_lo, tau_hi, [H] * U)
    assert [(a == v).sum() for v in (L, H, R)] == [42, 25, 17]
    exposure[7] = np.nan
    a, *_ = decide(dev, host, U, exposure, kappa, ebar, tau_lo, tau_hi, [H] * U)
    assert a[7] == R


def test_batched_phases_gate_exactly():
    """9 small units of mixed shapes / formats through CAPTURE, DECIDE, ENCODE, RECOVER."""
    rng = np.random.default_rng(1)
    shapes = [(96, 896), (64, 1536), (33, 4864), (128, 64), (40, 3584), (7, 18944), (256, 128), (64, 896), (50, 1536)]
    fmts = [api.FMT_E4M3FN_BLK, api.FMT_E4M3FN_RAW, api.FMT_INT8_BLK] * 3
    q = [L, L, L, H, H, H, R, R, H]                       # candidate plan
    want = [L, R, L, L, H, R, L, R, L]                    # desired actions before availability
    xs = [synth.activation_unit(rng, r, c) for r, c in shapes]
    bufs, units = [], []
    for x, (r, c), f in zip(xs, shapes, fmts):
        b = dict(x=G.dev(x), codes=G.Guarded(r * c), scales=G.Guarded(r * (c // 64) * 4), out=G.Guarded(r * c * 2),
                 rms=G.Guarded(r * 4))
        bufs.append(b)
        units.append(dict(x=b["x"], codes=b["codes"].ptr(), scales=None if f == api.FMT_E4M3FN_RAW else b["scales"].ptr(),
                          out=b["out"].ptr(), row_rms=b["rms"].ptr(), rows=r, cols=c, fmt=f,
                          block=0 if f == api.FMT_E4M3FN_RAW else 64))
    dev, host = api.make_unit_table(units)
    U = len(units)
    avail = G.dev(np.asarray(q, np.uint8))
    action = G.dev(np.asarray(want, np.uint8))
    rec = torch.zeros(U, dtype=torch.uint8, device="cuda")
    call = lambda phase: api.hilore_plan_apply(dev, host, U, phase, None, None, None, 0.0, 0.0, avail, action, None, rec, None)
    untouched = lambda g: bool((g.view == G.CANARY).all())

    call(api.PHASE_CAPTURE)
    for i, (x, f) in enumerate(zip(xs, fmts)):
        r, c = shapes[i]
        b = bufs[i]
        blk = 0 if f == api.FMT_E4M3FN_RAW else 64
        if q[i] == L:
            oc, osc = oracle.compress(x, f, blk)
            assert np.array_equal(b["codes"].numpy(np.uint8, (r, c)), oc)
            if blk:
                assert np.array_equal(b["scales"].numpy(np.float32, (r, c // 64)), osc)
        else:
            assert untouched(b["codes"]) and untouched(b["scales"])
        if q[i] in (L, H):
            assert G.rel_err(b["rms"].numpy(np.float32, (r,)), oracle.row_rms(x)).max() <= 1e-5
        else:
            assert untouched(b["rms"])
        assert np.array_equal(b["x"].cpu().numpy().view(np.uint16), x)      # forward keeps the original

    call(api.PHASE_DECIDE)
    a = action.cpu().numpy()
    assert a.tolist() == [L, R, L, L, H, R, R, R, L] and rec.cpu().numpy().tolist() == [int(v == R) for v in a]

    for b in bufs:
        b["rms"].view.fill_(G.CANARY)
    call(api.PHASE_ENCODE)                                 # q = H and action = L: units 3 and 8
    for i, (x, f) in enumerate(zip(xs, fmts)):
        r, c = shapes[i]
        blk = 0 if f == api.FMT_E4M3FN_RAW else 64
        if q[i] == H and a[i] == L:
            oc, osc = oracle.compress(x, f, blk)
            assert np.array_equal(bufs[i]["codes"].numpy(np.uint8, (r, c)), oc)
        elif q[i] != L:
            assert untouched(bufs[i]["codes"])
        assert untouched(bufs[i]["rms"])                   # token magnitudes are a capture-time product

    call(api.PHASE_RECOVER)
    for i, (x, f) in enumerate(zip(xs, fmts)):
        r, c = shapes[i]
        blk = 0 if f == api.FMT_E4M3FN_RAW else 64
        if a[i] == L:
            oc, osc = oracle.compress(x, f, blk)
            assert np.array_equal(bufs[i]["out"].numpy(np.uint16, (r, c)), oracle.recover(oc, osc, f, blk))
        else:
            assert untouched(bufs[i]["out"])               # H keeps its exact bundle, R is recomputed
        assert np.array_equal(bufs[i]["x"].cpu().numpy().view(np.uint16), x)


def test_units_without_buffers_are_skipped_and_bad_tables_rejected():
    x = synth.activation_unit(np.random.default_rng(2), 32, 128)
    xd = G.dev(x)
    units = [dict(x=xd, codes=None, scales=None, out=None, row_rms=None, rows=32, cols=128, fmt=api.FMT_E4M3FN_BLK, block=64)]
    dev, host = api.make_unit_table(units)
    avail, action = G.dev(np.array([L], np.uint8)), G.dev(np.array([L], np.uint8))
    for phase in (api.PHASE_CAPTURE, api.PHASE_ENCODE, api.PHASE_RECOVER):
        api.hilore_plan_apply(dev, host, 1, phase, None, None, None, 0, 0, avail, action, None, None, None)
    torch.cuda.synchronize()
    bad = [dict(units[0], cols=96)]
    d2, h2 = api.make_unit_table(bad)
    assert api.hilore_plan_apply(d2, h2, 1, api.PHASE_CAPTURE, None, None, None, 0, 0, avail, action, None, None, None,
                                 check=False) == api.SHAPE
    assert api.hilore_plan_apply(dev, host, 1, 9, None, None, None, 0, 0, avail, action, None, None, None,
                                 check=False) == api.INVALID_ARG


def test_tables_longer_than_one_launch_slice():
    """210 small units (more than the kernels stage per launch) with mixed formats and gates: CAPTURE then RECOVER
    must touch exactly the gated units, whichever slice of the table they fall into."""
    rng = np.random.default_rng(17)
    U = 210
    fmts = [(api.FMT_E4M3FN_BLK, api.FMT_E4M3FN_RAW, api.FMT_INT8_BLK)[i % 3] for i in range(U)]
    shapes = [((5, 64), (3, 192), (9, 128), (2, 1536))[i % 4] for i in range(U)]
    q = [(L, H, R, L, L)[i % 5] for i in range(U)]
    xs = [synth.activation_unit(rng, r, c) for r, c in shapes]
    bufs, units = [], []
    for x, (r, c), f in zip(xs, shapes, fmts):
        b = dict(x=G.dev(x), codes=G.Guarded(r * c), scales=G.Guarded(r * (c // 64) * 4), out=G.Guarded(r * c * 2),
                 rms=G.Guarded(r * 4))
        bufs.append(b)
        units.append(dict(x=b["x"], codes=b["codes"].ptr(), scales=None if f == api.FMT_E4M3FN_RAW else b["scales"].ptr(),
                          out=b["out"].ptr(), row_rms=b["rms"].ptr(), rows=r, cols=c, fmt=f,
                          block=0 if f == api.FMT_E4M3FN_RAW else 64))
    dev, host = api.make_unit_table(units)
    avail = G.dev(np.asarray(q, np.uint8))
    action = G.dev(np.asarray(q, np.uint8))                # every L candidate is decoded again
    api.hilore_plan_apply(dev, host, U, api.PHASE_CAPTURE, None, None, None, 0, 0, avail, action, None, None, None)
    api.hilore_plan_apply(dev, host, U, api.PHASE_RECOVER, None, None, None, 0, 0, avail, action, None, None, None)
    canary = G.CANARY | (G.CANARY << 8)
    for i, (x, (r, c), f, b) in enumerate(zip(xs, shapes, fmts, bufs)):
        blk = 0 if f == api.FMT_E4M3FN_RAW else 64
        codes, out, rms = b["codes"].numpy(np.uint8, (r, c)), b["out"].numpy(np.uint16, (r, c)), b["rms"].numpy(np.float32, (r,))
        if q[i] == L:
            oc, osc = oracle.compress(x, f, blk)
            assert np.array_equal(codes, oc), i
            if blk:
                assert np.array_equal(b["scales"].numpy(np.float32, (r, c // 64)), osc), i
            orec = oracle.recover(oc, osc, f, blk)
            nan = (orec & 0x7FFF) > 0x7F80
            assert np.array_equal(out[~nan], orec[~nan]), i
            assert G.rel_err(rms, oracle.row_rms(x)).max() <= 1e-5
        else:
            assert np.all(codes == G.CANARY) and np.all(out == canary), i
            if q[i] == H:
                assert G.rel_err(rms, oracle.row_rms(x)).max() <= 1e-5
            else:
                assert np.all(b["rms"].numpy(np.uint8, (r * 4,)) == G.CANARY), i
