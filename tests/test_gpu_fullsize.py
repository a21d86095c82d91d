"""Parity at the benchmark's full sizes and in its launch configuration.

The microbatch the benchmark times as its headline (7B-shaped, 24 GB) and two microbatches of the 1.5B-shaped step are
compared with the oracle WHOLE (its C calls spread over row ranges on the host cores).  Where a test samples instead
(the demotion run, the mixed table): a row's codes, scales, token RMS and reconstruction depend on that row only, so
the oracle can check any sample of rows.  Inputs are drawn on the device with the same recipe as the host generators
(N(0,1), 1 % of the channels x20)."""
import numpy as np
import pytest
import torch

import bench
import oracle
from paper_2609_33570_b200 import api, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu
R, H, L = api.ACT_R, api.ACT_H, api.ACT_L


def bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def check_rows(x, codes, scales, out, rms, rows, fmt, what=("codes", "rms", "out")):
    """Oracle check of the given row indices of one unit (device tensors)."""
    idx = torch.as_tensor(sorted(set(int(r) for r in rows)), device=x.device)
    xb = bits(x[idx])
    blk = 0 if fmt == api.FMT_E4M3FN_RAW else 64
    oc, osc = oracle.compress(xb, fmt, blk)
    if "codes" in what:
        assert np.array_equal(codes[idx].cpu().numpy(), oc)
        if blk:
            assert np.array_equal(scales[idx].cpu().numpy().view(np.uint32), osc.view(np.uint32))
    if "rms" in what:
        assert G.rel_err(rms[idx].cpu().numpy(), oracle.row_rms(xb)).max() <= 1e-5
    if "out" in what:
        assert np.array_equal(bits(out[idx]), oracle.recover(oc, osc, fmt, blk))


def sample_rows(rng, rows, n=24):
    return [0, 1, rows // 2, rows - 2, rows - 1] + rng.integers(0, rows, n).tolist()


def test_bench_step_1p5B_shaped_microbatch():
    """configs[1]: the exact object bench.py times (84 units, one launch per phase, all L)."""
    dev = torch.device("cuda", 0)
    cfg = bench.CONFIGS[2]
    wl = bench.Workload(api, synth, cfg, seed=0, device=dev)
    for t in wl.codes + wl.out:
        t.fill_(0xA5 if t.dtype == torch.uint8 else -1.0)
    wl.step(3)
    torch.cuda.synchronize()
    rng = np.random.default_rng(0)
    assert wl.action.cpu().tolist() == [L] * wl.U and wl.recompute.cpu().tolist() == [0] * wl.U
    want_bytes = [r * c + 4 * r * c // 64 for r, c in wl.shapes]
    assert wl.retained.cpu().tolist() == want_bytes
    for u in (0, 1, 2, 41, 42, 43, 81, 82, 83):
        check_rows(wl.x[u], wl.codes[u], wl.scales[u], wl.out[u], wl.rms[u], sample_rows(rng, wl.rows), api.FMT_E4M3FN_BLK)
    # coefficients of microbatch 3, then exposure, psi and action of a sample of units, every expected value from the
    # oracle's own chain (its omega, its token RMS of the whole unit): a unit's exposure depends on that unit only
    ro = wl.ro
    sl = slice(3 * cfg["mb_resp"], 4 * cfg["mb_resp"])
    adv = oracle.group_advantages(ro.rewards, ro.G)
    w, _, _ = oracle.grpo_coeffs(adv[sl], ro.logp_new[sl], ro.logp_old[sl], None, ro.mask[sl], N_norm=ro.n_valid)
    assert G.rel_err(wl.omega.cpu().numpy(), w).max() <= 1e-5
    sample = [0, 2, 41, 43, 83]
    o_rms = np.stack([oracle.row_rms(bits(wl.x[u])) for u in sample])
    oE, _ = oracle.unit_exposure(w, ro.mask[sl], o_rms)
    assert G.rel_err(wl.exposure.cpu().numpy()[sample], oE).max() <= 1e-5
    kappa, ebar = wl.kappa.cpu().numpy()[sample], wl.ebar.cpu().numpy()[sample]
    oa, opsi, orec, oret = oracle.plan(oE, kappa, ebar, float("inf"), float("inf"), [L] * len(sample), [wl.shapes[u][0] for u in sample],
                                       [wl.shapes[u][1] for u in sample], [1] * len(sample), [64] * len(sample))
    assert G.rel_err(wl.psi.cpu().numpy()[sample], opsi).max() <= 1e-5
    assert np.array_equal(wl.action.cpu().numpy()[sample], oa) and np.array_equal(wl.retained.cpu().numpy()[sample].view(np.uint64), oret)
    # every byte of every output was written: no canary left in a random sample of code rows
    for u in (5, 50):
        assert not bool((wl.scales[u] == 0).all())
    del wl
    torch.cuda.empty_cache()


def test_bench_step_7B_shaped_mixed_plan():
    """configs[2], the exact object bench.py times as its headline: 84 units [16384, 3584|3584|18944], capture with
    the candidate plan all H, `hilore_scores_plan` with the microbatch's thresholds (42 L / 25 H / 17 R), encode and
    recovery of the L units.  The WHOLE microbatch is compared: every expected value (token RMS of the 84 units,
    coefficients, exposure, psi, plan, retained bytes; codes, scales and reconstruction of the 42 L units) comes from
    the oracle's own chain on the host inputs, and every buffer of the other 42 units must be untouched."""
    dev = torch.device("cuda", 0)
    cfg = bench.CONFIGS[3]
    wl = bench.Workload(api, synth, cfg, seed=0, device=dev)
    wl.prepare_plan()
    for t in wl.codes:
        t.fill_(0xA5)
    for t in wl.scales:
        t.fill_(-7.0)
    for t in wl.out:
        t.fill_(-3.0)
    mb = 5
    wl.step(mb)
    torch.cuda.synchronize()
    a = wl.action.cpu().numpy()
    assert np.array_equal(a, wl.expected_action[mb]) and [(a == v).sum() for v in (L, H, R)] == [42, 25, 17]
    assert np.array_equal(wl.recompute.cpu().numpy(), (a == R).astype(np.uint8))
    ro = wl.ro
    sl = slice(mb * cfg["mb_resp"], (mb + 1) * cfg["mb_resp"])
    adv = oracle.group_advantages(ro.rewards, ro.G)
    w, _, _ = oracle.grpo_coeffs(adv[sl], ro.logp_new[sl], ro.logp_old[sl], None, ro.mask[sl], N_norm=ro.n_valid)
    assert G.rel_err(wl.omega.cpu().numpy(), w).max() <= 1e-5
    # all 84 units: token RMS, exposure, psi, action and retained bytes from the oracle's chain
    from concurrent.futures import ThreadPoolExecutor
    U = wl.U
    with ThreadPoolExecutor(8) as pool:
        o_rms = np.stack(list(pool.map(lambda u: oracle.row_rms(bits(wl.x[u])), range(U))))
    assert G.rel_err(wl.rms.cpu().numpy(), o_rms).max() <= 1e-5
    oE, _ = oracle.unit_exposure(w, ro.mask[sl], o_rms)
    assert G.rel_err(wl.exposure.cpu().numpy(), oE).max() <= 1e-5
    kappa, ebar = wl.kappa.cpu().numpy(), wl.ebar.cpu().numpy()
    oa, opsi, orec, oret = oracle.plan(oE, kappa, ebar, wl.tau[mb][0], wl.tau[mb][1], [H] * U, [sh[0] for sh in wl.shapes],
                                       [sh[1] for sh in wl.shapes], [1] * U, [64] * U)
    assert G.rel_err(wl.psi.cpu().numpy(), opsi).max() <= 1e-5
    assert np.array_equal(a, oa) and np.array_equal(wl.retained.cpu().numpy().view(np.uint64), oret)
    # every unit assigned L, whole: codes, scale bits and reconstruction are the oracle's
    for u in range(U):
        if a[u] == L:
            oc, osc, oout, _ = oracle_unit(bits(wl.x[u]))
            assert np.array_equal(wl.codes[u].cpu().numpy(), oc)
            assert np.array_equal(wl.scales[u].cpu().numpy().view(np.uint32), osc.view(np.uint32))
            assert np.array_equal(bits(wl.out[u]), oout)
        else:                                                 # H keeps its bundle, R is recomputed: nothing written
            assert bool((wl.codes[u] == 0xA5).all()) and bool((wl.scales[u] == -7.0).all())
            assert bool((wl.out[u] == -3.0).all())
    del wl
    torch.cuda.empty_cache()


def test_7B_shaped_mixed_plan():
    """configs[2]: 84 units [16384, 3584|3584|18944], candidate plan all H, thresholds at the 50 % / 70 %
    quantiles of psi (42 L / 17 R / 25 H), post-forward encode and recovery of the L units only."""
    dev = torch.device("cuda", 0)
    rows, layers = 16384, 28
    shapes = synth.layer_unit_shapes("7B", rows, layers)
    U = len(shapes)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1)
    x = [synth.activation_unit_device(gen, r, c, dev) for r, c in shapes]
    codes = [torch.full((r, c), 0xA5, dtype=torch.uint8, device=dev) for r, c in shapes]
    scales = [torch.full((r, c // 64), -7.0, dtype=torch.float32, device=dev) for r, c in shapes]
    out = [torch.full((r, c), -3.0, dtype=torch.bfloat16, device=dev) for r, c in shapes]   # no two units share a buffer
    rms = torch.full((U, rows), -1.0, dtype=torch.float32, device=dev)
    units = [dict(x=x[i], codes=codes[i], scales=scales[i], out=out[i],
                  row_rms=rms[i], rows=r, cols=c, fmt=api.FMT_E4M3FN_BLK, block=64) for i, (r, c) in enumerate(shapes)]
    udev, uhost = api.make_unit_table(units, dev)
    avail = torch.full((U,), H, dtype=torch.uint8, device=dev)
    action = torch.zeros(U, dtype=torch.uint8, device=dev)
    rec = torch.zeros(U, dtype=torch.uint8, device=dev)
    retained = torch.zeros(U, dtype=torch.int64, device=dev)
    psi = torch.zeros(U, dtype=torch.float32, device=dev)
    expo = torch.zeros(U, dtype=torch.float32, device=dev)
    call = lambda phase, **k: api.hilore_plan_apply(udev, uhost, U, phase, k.get("E"), k.get("kappa"), k.get("ebar"),
                                                    k.get("lo", 0.0), k.get("hi", 0.0), avail, action, k.get("psi"), rec,
                                                    retained)
    call(api.PHASE_CAPTURE)                                   # q = H everywhere: token RMS only
    torch.cuda.synchronize()
    assert all(bool((c[:2] == 0xA5).all()) for c in codes[:6])
    # microbatch 5 of 256: 8 responses x 2048 slots; G = 16, so a prompt group spans two microbatches
    ro = synth.rollout(2, 16, 16, 2048)
    mb, n_mb = 5, 8
    sl = slice(mb * n_mb, (mb + 1) * n_mb)
    t = lambda a: torch.from_numpy(a).to(dev)
    omega = torch.empty((n_mb, 2048), dtype=torch.float32, device=dev)
    api.hilore_grpo_coeffs(t(ro.rewards), ro.n_resp, 16, mb * n_mb, n_mb, 2048, t(ro.logp_new[sl]), t(ro.logp_old[sl]), None,
                           t(ro.mask[sl]), 2048 * 128 * 16, None, 0.2, 0.0, 1e-6, None, omega, None, None)
    nws = api.hilore_workspace_bytes(U, rows)
    ws = torch.empty(nws, dtype=torch.uint8, device=dev)
    api.hilore_unit_exposure(omega, t(ro.mask[sl]), n_mb, 2048, rms, U, rows, 0, 1e-8, expo, None, ws, nws)
    kappa = torch.from_numpy(np.random.default_rng(3).uniform(0.5, 2.0, U).astype(np.float32)).to(dev)
    ebar = torch.full((U,), 0.0266, dtype=torch.float32, device=dev)
    # thresholds at midpoints between order statistics of psi, so that no unit sits near a threshold
    E = expo.cpu().numpy()
    psi_h = (kappa.cpu().numpy() * E).astype(np.float32) * ebar.cpu().numpy()
    srt = np.sort(psi_h)
    lo, hi = float((srt[41] + srt[42]) / 2), float((srt[U - 26] + srt[U - 25]) / 2)
    call(api.PHASE_DECIDE, E=expo, kappa=kappa, ebar=ebar, lo=lo, hi=hi, psi=psi)
    a = action.cpu().numpy()
    assert [(a == v).sum() for v in (L, H, R)] == [42, 25, 17]
    assert np.array_equal(rec.cpu().numpy(), (a == R).astype(np.uint8))
    # expected values of a sample of units from the oracle's own chain: its advantages and omega from the host
    # inputs, its token RMS of the whole unit, its exposure, psi and action
    adv_o = oracle.group_advantages(ro.rewards, 16)
    w_o, _, _ = oracle.grpo_coeffs(adv_o[sl], ro.logp_new[sl], ro.logp_old[sl], None, ro.mask[sl], N_norm=2048 * 128 * 16)
    assert G.rel_err(omega.cpu().numpy(), w_o).max() <= 1e-5
    sample = [0, 1, 40, 82, 5]                             # four narrow units and one wide one
    o_rms = np.stack([oracle.row_rms(bits(x[u])) for u in sample])
    oE, _ = oracle.unit_exposure(w_o, ro.mask[sl], o_rms)
    assert G.rel_err(E[sample], oE).max() <= 1e-5
    oa, opsi, orec, oret = oracle.plan(oE, kappa.cpu().numpy()[sample], ebar.cpu().numpy()[sample], lo, hi, [H] * len(sample),
                                       [shapes[u][0] for u in sample], [shapes[u][1] for u in sample], [1] * len(sample),
                                       [64] * len(sample))
    assert G.rel_err(psi.cpu().numpy()[sample], opsi).max() <= 1e-5
    assert np.array_equal(a[sample], oa) and np.array_equal(rec.cpu().numpy()[sample], orec)
    assert np.array_equal(retained.cpu().numpy()[sample].view(np.uint64), oret)
    call(api.PHASE_ENCODE)
    call(api.PHASE_RECOVER)
    torch.cuda.synchronize()
    rng = np.random.default_rng(4)
    narrow_L = [u for u in range(U) if a[u] == L and shapes[u][1] < 10000]
    wide_L = [u for u in range(U) if a[u] == L and shapes[u][1] > 10000]
    for u in narrow_L[:3] + narrow_L[-2:]:
        check_rows(x[u], codes[u], scales[u], out[u], rms[u], sample_rows(rng, rows, 12), api.FMT_E4M3FN_BLK)
    for u in wide_L[:2] + wide_L[-1:]:
        check_rows(x[u], codes[u], scales[u], out[u], rms[u], sample_rows(rng, rows, 8), api.FMT_E4M3FN_BLK)
    for u in [v for v in range(U) if a[v] != L][:8]:          # H keeps its bundle, R is recomputed: nothing written
        assert bool((codes[u] == 0xA5).all()) and bool((scales[u] == -7.0).all())
        assert bool((out[u] == -3.0).all())
        check_rows(x[u], None, None, None, rms[u], sample_rows(rng, rows, 6), api.FMT_E4M3FN_BLK, what=("rms",))
    del x, codes, scales, out
    torch.cuda.empty_cache()


def test_variable_length_rollout_batch_full_size():
    """configs[3]: 256 prompts x G=8 x 4096 slots, lengths U{128..4096}, rewards U[0,1), 13 equal-reward groups."""
    ro = synth.rollout(0, 256, 8, 4096, rewards="uniform", lengths="uniform", equal_group_fraction=0.05)
    got = G.grpo_coeffs(ro, N_on_device=True, extras=False)
    assert got["N"] == ro.n_valid
    adv = oracle.group_advantages(ro.rewards, 8)
    w, r, chi = oracle.grpo_coeffs(adv, ro.logp_new, ro.logp_old, None, ro.mask, N_norm=ro.n_valid)
    hi, lo = np.float32(1.2), np.float32(0.8)
    near = (np.abs(r - hi) <= 4 * np.spacing(hi)) | (np.abs(r - lo) <= 4 * np.spacing(lo))
    assert G.rel_err(got["omega"][~near], w[~near]).max() <= 1e-5
    assert near.sum() < 50
    Rg = ro.rewards.reshape(-1, 8)
    eq = np.where(Rg.max(axis=1) == Rg.min(axis=1))[0]
    assert len(eq) == 13
    for g in eq:
        assert np.all(got["omega"][g * 8:(g + 1) * 8] == 0)
    assert np.all(got["omega"][ro.mask == 0] == 0)
    # one microbatch of 4 responses: masked exposure over a [16384, 3584] unit's token RMS
    rng = np.random.default_rng(1)
    x = synth.activation_unit(rng, 16384, 3584)
    _, _, rms = G.compress(x, api.FMT_E4M3FN_BLK)
    om = np.ascontiguousarray(got["omega"][8:12])
    E, sw = G.unit_exposure(om, np.ascontiguousarray(ro.mask[8:12]), rms[None, :])
    oE, osw = oracle.unit_exposure(np.ascontiguousarray(w[8:12]), np.ascontiguousarray(ro.mask[8:12]), oracle.row_rms(x)[None, :])
    assert G.rel_err(E, oE).max() <= 1e-5 and abs(sw - osw) <= 1e-5 * osw


def test_4GiB_unit_uses_64_bit_offsets():
    """configs[4], top end: one unit of 2^31 elements ([524288, 4096] bf16 = 4 GiB), both formats, compared WHOLE: the
    unit is a 128 MiB block of rows repeated 32 times with two rows changed, so the oracle's result for the block (and
    for the two rows) gives every expected byte."""
    dev = torch.device("cuda", 0)
    rows, cols = 1 << 19, 4096
    gen = torch.Generator(device=dev)
    gen.manual_seed(5)
    base = synth.activation_unit_device(gen, 1 << 14, cols, dev)
    reps = rows // base.shape[0]
    x = base.repeat(reps, 1)
    changed = [rows - 1, rows // 2 + 1]
    x[-1, -64:] = 3.0            # make the very last block distinctive
    x[rows // 2 + 1, :64] = -5.0
    for fmt in (api.FMT_E4M3FN_BLK, api.FMT_E4M3FN_RAW):
        blk = 64 if fmt == api.FMT_E4M3FN_BLK else 0
        codes = torch.full((rows, cols), 0xA5, dtype=torch.uint8, device=dev)
        scales = torch.full((rows, cols // 64), -7.0, dtype=torch.float32, device=dev) if blk else None
        rms = torch.full((rows,), -1.0, dtype=torch.float32, device=dev)
        out = torch.full((rows, cols), -3.0, dtype=torch.bfloat16, device=dev)
        api.hilore_compress(x, rows, cols, cols, fmt, blk, codes, scales, rms)
        api.hilore_recover(codes, scales, rows, cols, fmt, blk, out, cols)
        torch.cuda.synchronize()
        oc, osc, oout, orms = oracle_unit(bits(base), fmt=fmt)
        want_codes = torch.from_numpy(oc).to(dev).repeat(reps, 1)
        want_out = torch.from_numpy(oout.view(np.int16)).to(dev).repeat(reps, 1)
        want_rms = torch.from_numpy(orms).to(dev).repeat(reps)
        want_scales = torch.from_numpy(osc.view(np.int32)).to(dev).repeat(reps, 1) if blk else None
        for r in changed:                                     # the two rows that differ from the block
            rc, rs, ro_, rr = oracle_unit(bits(x[r:r + 1]), threads=1, fmt=fmt)
            want_codes[r] = torch.from_numpy(rc[0]).to(dev)
            want_out[r] = torch.from_numpy(ro_.view(np.int16)[0]).to(dev)
            want_rms[r] = float(rr[0])
            if blk:
                want_scales[r] = torch.from_numpy(rs.view(np.int32)[0]).to(dev)
        assert torch.equal(codes, want_codes)
        assert torch.equal(out.view(torch.int16), want_out)
        if blk:
            assert torch.equal(scales.view(torch.int32), want_scales)
        err = ((rms.double() - want_rms.double()).abs() / want_rms.double().abs().clamp_min(1e-300)).max().item()
        assert err <= 1e-5
        del codes, scales, rms, out, want_codes, want_out, want_rms, want_scales
        torch.cuda.empty_cache()


def xor_fold(t: torch.Tensor) -> int:
    """xor of all 64-bit words of a device tensor (its byte size must be a multiple of 8)."""
    w = t.contiguous().view(torch.uint8).view(-1).view(torch.int64)
    while w.numel() > 1:
        h = w.numel() // 2
        rest = w[2 * h:]
        w = torch.bitwise_xor(w[:h], w[h:2 * h])
        if rest.numel():
            w = torch.cat([w, rest])
    return int(w.item())


def xor_fold_host(a: np.ndarray) -> int:
    return int(np.bitwise_xor.reduce(np.ascontiguousarray(a).view(np.int64).reshape(-1)))


def oracle_unit(xb: np.ndarray, threads=16, fmt=None):
    """Codes, scales, reconstruction and token RMS of a whole unit from the oracle, its C calls spread over row ranges."""
    from concurrent.futures import ThreadPoolExecutor
    fmt = oracle.FMT_E4M3FN_BLK if fmt is None else fmt
    blk = 0 if fmt == oracle.FMT_E4M3FN_RAW else 64
    threads = max(1, min(threads, xb.shape[0]))
    cuts = [xb.shape[0] * i // threads for i in range(threads + 1)]

    def part(ab):
        x = np.ascontiguousarray(xb[ab[0]:ab[1]])
        c, s = oracle.compress(x, fmt, blk)
        return c, s, oracle.recover(c, s, fmt, blk), oracle.row_rms(x)
    with ThreadPoolExecutor(threads) as pool:
        parts = list(pool.map(part, zip(cuts[:-1], cuts[1:])))
    return tuple(np.concatenate([p[i] for p in parts]) if parts[0][i] is not None else None for i in range(4))


@pytest.mark.parametrize("rows,cols", [(16384, 18944), (36000, 4096), (20001, 8960)])
def test_whole_units_that_are_shared_in_several_windows(rows, cols):
    """Single units large enough to be cut into windows (rows of 37 KB, 8 KB and 17.5 KB; the last two with row counts
    that leave uneven last windows), compared WHOLE with the oracle: compress with token RMS (row shares), compress
    without it and recover (16 KB pieces).  A row or piece lost or done twice at a window or CTA boundary shows here."""
    dev = torch.device("cuda", 0)
    gen = torch.Generator(device=dev)
    gen.manual_seed(rows + cols)
    x = synth.activation_unit_device(gen, rows, cols, dev)
    oc, osc, oout, orms = oracle_unit(bits(x))
    for with_rms in (True, False):
        codes = torch.full((rows, cols), 0xA5, dtype=torch.uint8, device=dev)
        scales = torch.full((rows, cols // 64), -7.0, dtype=torch.float32, device=dev)
        rms = torch.full((rows,), -1.0, dtype=torch.float32, device=dev)
        out = torch.full((rows, cols), -3.0, dtype=torch.bfloat16, device=dev)
        api.hilore_compress(x, rows, cols, cols, api.FMT_E4M3FN_BLK, 64, codes, scales, rms if with_rms else None)
        api.hilore_recover(codes, scales, rows, cols, api.FMT_E4M3FN_BLK, 64, out, cols)
        torch.cuda.synchronize()
        assert np.array_equal(codes.cpu().numpy(), oc)
        assert np.array_equal(scales.cpu().numpy().view(np.uint32), osc.view(np.uint32))
        assert np.array_equal(bits(out), oout)
        if with_rms:
            assert G.rel_err(rms.cpu().numpy(), orms).max() <= 1e-5
        else:
            assert bool((rms == -1.0).all())
        del codes, scales, rms, out
    torch.cuda.empty_cache()


def test_1p5B_shaped_whole_units_and_checksums_over_microbatches():
    """configs[1]: the step bench.py's 1.5B-shaped leg times, on fresh activations per microbatch.  Microbatches 0 and
    63: all 84 units compared WHOLE with the oracle (codes, scale bits, reconstruction, token RMS), and their xor-folds
    with the oracle's.  Eight microbatches: xor-fold of the codes and scale bits of all 84 units,
    equal between two runs on the same inputs (same bits whatever the scheduling) and different between microbatches."""
    dev = torch.device("cuda", 0)
    cfg = bench.CONFIGS[2]
    wl = bench.Workload(api, synth, cfg, seed=0, device=dev)
    mbs = [0, 9, 18, 27, 36, 45, 54, 63]

    def run(mb, check_whole):
        gen = torch.Generator(device=dev)
        gen.manual_seed(1000 + mb)
        for i, (r, c) in enumerate(wl.shapes):
            wl.x[i].copy_(synth.activation_unit_device(gen, r, c, dev))
        for t in wl.codes + wl.scales:
            t.fill_(0)
        wl.step(mb)
        torch.cuda.synchronize()
        sums = [(xor_fold(wl.codes[u]), xor_fold(wl.scales[u])) for u in range(wl.U)]
        if check_whole:
            for u in range(wl.U):                                # all 84 units of the microbatch, whole
                oc, osc, oout, orms = oracle_unit(bits(wl.x[u]))
                assert np.array_equal(wl.codes[u].cpu().numpy(), oc)
                assert np.array_equal(wl.scales[u].cpu().numpy().view(np.uint32), osc.view(np.uint32))
                assert np.array_equal(bits(wl.out[u]), oout)
                assert G.rel_err(wl.rms[u].cpu().numpy(), orms).max() <= 1e-5
                assert sums[u] == (xor_fold_host(oc), xor_fold_host(osc))
        return sums

    first = {mb: run(mb, mb in (0, 63)) for mb in mbs}
    again = {mb: run(mb, False) for mb in mbs}
    assert first == again
    assert len({tuple(v) for v in first.values()}) == len(mbs)
    del wl
    torch.cuda.empty_cache()


def test_7B_shaped_plan_with_demoted_candidates():
    """configs[2], second run: a quarter of the units captured as L candidates, a quarter as R candidates, the rest H,
    through CAPTURE / DECIDE / ENCODE / RECOVER at full size.  Desired actions outside a unit's candidate set are
    demoted to R; R candidates are never touched; H candidates assigned L are encoded after the forward pass."""
    dev = torch.device("cuda", 0)
    rows, layers = 16384, 28
    shapes = synth.layer_unit_shapes("7B", rows, layers)
    U = len(shapes)
    gen = torch.Generator(device=dev)
    gen.manual_seed(11)
    x = [synth.activation_unit_device(gen, r, c, dev) for r, c in shapes]
    codes = [torch.full((r, c), 0xA5, dtype=torch.uint8, device=dev) for r, c in shapes]
    scales = [torch.full((r, c // 64), -7.0, dtype=torch.float32, device=dev) for r, c in shapes]
    out = [torch.full((r, c), -3.0, dtype=torch.bfloat16, device=dev) for r, c in shapes]
    rms = torch.full((U, rows), -1.0, dtype=torch.float32, device=dev)
    units = [dict(x=x[i], codes=codes[i], scales=scales[i], out=out[i], row_rms=rms[i], rows=r, cols=c,
                  fmt=api.FMT_E4M3FN_BLK, block=64) for i, (r, c) in enumerate(shapes)]
    udev, uhost = api.make_unit_table(units, dev)
    q = np.array([(L, H, R, H)[i % 4] for i in range(U)], dtype=np.uint8)     # 21 L, 21 R, 42 H, every width in each
    assert [(q == v).sum() for v in (L, R, H)] == [21, 21, 42]
    avail = torch.from_numpy(q).to(dev)
    action = torch.zeros(U, dtype=torch.uint8, device=dev)
    rec = torch.zeros(U, dtype=torch.uint8, device=dev)
    retained = torch.zeros(U, dtype=torch.int64, device=dev)
    psi = torch.zeros(U, dtype=torch.float32, device=dev)
    expo = torch.zeros(U, dtype=torch.float32, device=dev)
    call = lambda phase, **k: api.hilore_plan_apply(udev, uhost, U, phase, k.get("E"), k.get("kappa"), k.get("ebar"),
                                                    k.get("lo", 0.0), k.get("hi", 0.0), avail, action, k.get("psi"), rec,
                                                    retained)
    call(api.PHASE_CAPTURE)
    torch.cuda.synchronize()
    rms_h = rms.cpu().numpy()
    for u in range(U):                                      # R candidates: nothing written; H: token RMS only
        if q[u] == R:
            assert np.all(rms_h[u] == -1.0) and bool((codes[u][::4097] == 0xA5).all())
        elif q[u] == H:
            assert np.all(rms_h[u] > 0) and bool((codes[u] == 0xA5).all()) and bool((scales[u] == -7.0).all())
        else:
            assert np.all(rms_h[u] > 0) and not bool((scales[u] == -7.0).any())
    ro = synth.rollout(12, 16, 16, 2048)
    mb, n_mb = 3, 8
    sl = slice(mb * n_mb, (mb + 1) * n_mb)
    t = lambda a: torch.from_numpy(a).to(dev)
    omega = torch.empty((n_mb, 2048), dtype=torch.float32, device=dev)
    nws = api.hilore_workspace_bytes(U, rows)
    ws = torch.empty(nws, dtype=torch.uint8, device=dev)
    rms.clamp_(min=0.0)                                     # R candidates have no token RMS: a defined value for the score
    api.hilore_coeffs_exposure(t(ro.rewards), ro.n_resp, 16, mb * n_mb, n_mb, 2048, t(ro.logp_new[sl]), t(ro.logp_old[sl]),
                               None, t(ro.mask[sl]), ro.n_valid, None, 0.2, 0.0, 1e-6, rms, U, rows, 0, 1e-8, omega, expo,
                               None, ws, nws)
    kappa = np.random.default_rng(13).uniform(0.5, 2.0, U).astype(np.float32)
    ebar = np.full(U, 0.0266, dtype=np.float32)
    E = expo.cpu().numpy()
    psi_h = (kappa * E).astype(np.float32) * ebar
    live = np.sort(psi_h[q != R])
    lo, hi = float((live[30] + live[31]) / 2), float((live[44] + live[45]) / 2)
    call(api.PHASE_DECIDE, E=expo, kappa=t(kappa), ebar=t(ebar), lo=lo, hi=hi, psi=psi)
    a = action.cpu().numpy()
    # the plan from the oracle on the same exposure bits (a unit's action depends on its own psi only)
    oa, opsi, orec, oret = oracle.plan(E, kappa, ebar, lo, hi, q, [s[0] for s in shapes], [s[1] for s in shapes], [1] * U, [64] * U)
    assert np.array_equal(a, oa) and np.array_equal(rec.cpu().numpy(), orec)
    assert np.array_equal(psi.cpu().numpy().view(np.uint32), opsi.view(np.uint32))
    assert np.array_equal(retained.cpu().numpy().view(np.uint64), oret)
    assert np.all(a[q == R] == R) and np.all(a[(q == L)] != H)                 # demotion
    assert ((q == L) & (a == R)).sum() > 0 and ((q == H) & (a == L)).sum() > 0  # both kinds occur in this draw
    codes_before = {u: xor_fold(codes[u]) for u in range(U) if q[u] == L}
    call(api.PHASE_ENCODE)
    call(api.PHASE_RECOVER)
    torch.cuda.synchronize()
    rng = np.random.default_rng(14)
    enc = [u for u in range(U) if q[u] == H and a[u] == L]
    cap = [u for u in range(U) if q[u] == L and a[u] == L]
    for u in enc[:3] + enc[-2:] + cap[:2] + cap[-1:]:
        check_rows(x[u], codes[u], scales[u], out[u], rms[u], sample_rows(rng, rows, 10), api.FMT_E4M3FN_BLK)
    for u in codes_before:                                   # ENCODE leaves the units captured as L alone
        assert xor_fold(codes[u]) == codes_before[u]
    for u in range(U):
        if a[u] != L:                                       # nothing decoded into units that are not L
            assert bool((out[u][::257] == -3.0).all())
        if q[u] == R or (q[u] == H and a[u] != L):          # never compressed
            assert bool((codes[u] == 0xA5).all()) and bool((scales[u] == -7.0).all())
    del x, codes, scales, out
    torch.cuda.empty_cache()
