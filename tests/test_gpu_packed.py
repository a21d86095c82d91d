"""Parity of the packed-layout coefficient and exposure calls with the oracle (fp32 within 1e-5 relative; the clip
indicator exact away from the clip bounds), and equality with the dense kernels on the same tokens."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_33570_b200 import api, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu
RTOL = 1e-5


def dev_i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


def packed_gpu(ro, pk, beta=0.0, N=None, resp_offset=0, n_on_device=False):
    n_seq, n_tok = len(pk.rows), pk.n_tok
    adv, omega = G.Guarded(max(n_seq, 1) * 4), G.Guarded(n_tok * 4)
    ratio, chi = G.Guarded(n_tok * 4), G.Guarded(n_tok)
    mask = G.dev(pk.mask)
    ndev = None
    if n_on_device:
        ndev = torch.zeros(1, dtype=torch.int64, device="cuda")
        api.hilore_mask_count(mask, n_tok, ndev)
    api.hilore_grpo_coeffs_packed(G.dev(ro.rewards), ro.n_resp, ro.G, resp_offset, n_seq, dev_i32(pk.cu_seqlens), n_tok,
                                  G.dev(pk.logp_new), G.dev(pk.logp_old), G.dev(pk.logp_ref) if beta else None, mask,
                                  0 if n_on_device else (ro.n_valid if N is None else N), ndev, 0.2, beta, 1e-6, adv.ptr(),
                                  omega.ptr(), ratio.ptr(), chi.ptr())
    return (adv.numpy(np.float32, (n_seq,)), omega.numpy(np.float32, (n_tok,)), ratio.numpy(np.float32, (n_tok,)),
            chi.numpy(np.uint8, (n_tok,)))


def check(ro, pk, got, beta, N):
    adv, omega, ratio, chi = got
    adv_o = oracle.group_advantages(ro.rewards, ro.G)[pk.rows]
    w, r, c = oracle.grpo_coeffs_packed(adv_o, pk.cu_seqlens, pk.logp_new, pk.logp_old, pk.logp_ref if beta else None,
                                        pk.mask, N_norm=N, beta=beta)
    lens = np.diff(pk.cu_seqlens)
    assert G.rel_err(adv, adv_o).max(initial=0) <= RTOL and np.array_equal(adv == 0, adv_o == 0)
    hi, lo = np.float32(1.2), np.float32(0.8)
    near = (np.abs(r - hi) <= 4 * np.spacing(hi)) | (np.abs(r - lo) <= 4 * np.spacing(lo))
    assert not np.any((chi != c) & ~near)
    assert G.rel_err(ratio, r).max(initial=0) <= RTOL
    ok = ~near
    err = G.rel_err(omega[ok], w[ok])
    kl = beta * pk.mask / N * (1 - np.exp(pk.logp_ref.astype(np.float64) - pk.logp_new))
    floor = RTOL * np.maximum(np.abs(w.astype(np.float64) - kl), np.abs(kl))[ok]
    assert np.all((err <= RTOL) | (np.abs(omega[ok].astype(np.float64) - w[ok]) <= floor))
    assert np.all(omega[pk.mask == 0] == 0)
    return lens


@pytest.mark.parametrize("beta", [0.0, 1e-3])
@pytest.mark.parametrize("P,G_,T,max_prompt", [(8, 8, 700, 300), (3, 4, 36, 5), (64, 16, 64, 3)])
def test_packed_coeffs_match_oracle(P, G_, T, max_prompt, beta):
    ro = synth.rollout(31, P, G_, T, lengths="uniform", min_len=1, rewards="bernoulli", equal_group_fraction=0.25)
    ro.logp_old[:] = ro.logp_new + np.random.default_rng(4).normal(0, 0.12, ro.logp_new.shape).astype(np.float32)
    pk = synth.pack_rollout(ro, 6, max_prompt=max_prompt)
    got = packed_gpu(ro, pk, beta=beta)
    check(ro, pk, got, beta, ro.n_valid)
    # the same tokens through the dense kernel: identical bits (same arithmetic per token)
    dense = G.grpo_coeffs(ro, N_norm=ro.n_valid, beta=beta)
    seq = np.repeat(np.arange(len(pk.rows)), np.diff(pk.cu_seqlens))
    resp = pk.dense_t >= 0
    i, t = pk.rows[seq[resp]], pk.dense_t[resp]
    assert np.array_equal(got[1][resp], dense["omega"][i, t])
    assert np.array_equal(got[2][resp], dense["ratio"][i, t])


def test_packed_microbatch_slice_device_normaliser_and_empty_sequences():
    ro = synth.rollout(32, 4, 8, 128, lengths="uniform", min_len=2)
    rows = np.arange(8, 24)                                  # a microbatch: responses 8..23 of the rollout batch
    pk = synth.pack_rollout(ro, 2, rows=rows, max_prompt=17)
    # insert empty sequences by repeating boundaries: sequences 3 and 9 own nothing
    lens = np.diff(pk.cu_seqlens).astype(np.int64)
    keep = np.ones(len(rows), bool)
    keep[[3, 9]] = False
    cu2 = np.zeros(len(rows) + 1, np.int64)
    np.cumsum(np.where(keep, lens, 0), out=cu2[1:])
    sel = np.concatenate([np.arange(pk.cu_seqlens[j], pk.cu_seqlens[j + 1]) for j in range(len(rows)) if keep[j]])
    pk2 = synth.PackedRollout(cu2.astype(np.int32), rows, pk.logp_new[sel].copy(), pk.logp_old[sel].copy(),
                              pk.logp_ref[sel].copy(), pk.mask[sel].copy(), pk.dense_t[sel].copy())
    N = int(pk2.mask.sum())
    got = packed_gpu(ro, pk2, beta=1e-3, resp_offset=8, n_on_device=True)
    check(ro, pk2, got, 1e-3, N)


@pytest.mark.parametrize("beta", [0.0, 1e-3])
@pytest.mark.parametrize("tail", [0, 3, 13])
def test_packed_tiny_empty_and_long_sequences_in_one_microbatch(beta, tail):
    """The warp-tile kernel's cases in one microbatch: runs of sequences of 0-13 tokens (more than 32 sequence starts
    inside one 512-token tile, boundaries inside a lane's eight tokens, empty sequences), long sequences that span
    several tiles, and a token count that is not a multiple of eight (outputs between canaries).  Against the oracle,
    and bit for bit against the generic kernel, which the same call takes when a tensor is only 16-byte aligned."""
    rng = np.random.default_rng(77 + tail)
    G_ = 8
    lens = np.concatenate([rng.choice([0, 0, 1, 2, 3, 5, 8, 13], 400), rng.integers(600, 1500, 9), rng.choice([0, 1, 7, 9], 150),
                           rng.integers(600, 1500, 8), rng.choice([0, 2, 8, 16], 57)])
    rng.shuffle(lens[:409])
    lens[-1] += (tail - int(lens.sum())) % 8                  # token count = tail (mod 8)
    n_seq = len(lens)
    assert n_seq % G_ == 0
    ro = synth.rollout(5, n_seq // G_, G_, 4, rewards="bernoulli", equal_group_fraction=0.2)
    n_tok = int(lens.sum())
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    lp = rng.normal(-1.5, 0.5, n_tok).astype(np.float32)
    pk = synth.PackedRollout(cu, np.arange(n_seq), lp, (lp + rng.normal(0, 0.12, n_tok)).astype(np.float32),
                             (lp + rng.normal(0, 0.1, n_tok)).astype(np.float32), (rng.random(n_tok) < 0.8).astype(np.uint8),
                             np.zeros(n_tok, np.int64))
    N = int(pk.mask.sum())
    got = packed_gpu(ro, pk, beta=beta, N=N)
    check(ro, pk, got, beta, N)

    def shifted(a, dtype):                                  # the same values at an address that is 16 mod 32 (masks: 4 mod 8)
        t = torch.zeros(len(a) + 64, dtype=dtype, device="cuda")
        off = 4 + (-(t.data_ptr() // 4) % 8 if dtype == torch.float32 else -t.data_ptr() % 8)
        v = t[off:off + len(a)]
        v.copy_(torch.from_numpy(np.ascontiguousarray(a)))
        return v
    ln, lo, lr, mk = shifted(pk.logp_new, torch.float32), shifted(pk.logp_old, torch.float32), shifted(pk.logp_ref, torch.float32), \
        shifted(pk.mask, torch.uint8)
    assert ln.data_ptr() % 32 == 16 and mk.data_ptr() % 8 == 4
    adv = torch.zeros(n_seq, device="cuda")
    omega, ratio = shifted(np.zeros(n_tok, np.float32), torch.float32), shifted(np.zeros(n_tok, np.float32), torch.float32)
    chi = shifted(np.zeros(n_tok, np.uint8), torch.uint8)
    api.hilore_grpo_coeffs_packed(G.dev(ro.rewards), ro.n_resp, ro.G, 0, n_seq, dev_i32(cu), n_tok, ln, lo, lr if beta else None,
                                  mk, N, None, 0.2, beta, 1e-6, adv, omega, ratio, chi)
    torch.cuda.synchronize()
    assert np.array_equal(adv.cpu().numpy().view(np.uint32), got[0].view(np.uint32))
    assert np.array_equal(omega.cpu().numpy().view(np.uint32), got[1].view(np.uint32))
    assert np.array_equal(ratio.cpu().numpy().view(np.uint32), got[2].view(np.uint32))
    assert np.array_equal(chi.cpu().numpy(), got[3])


def test_packed_coefficients_of_a_whole_rollout_batch_of_2p24_tokens():
    """The largest point of the sweep on this layout: 2^24 + 5 tokens in about 8200 sequences of 1-3 K tokens (with a
    few empty ones and a run of very short ones), every token against the oracle, with the K3 term."""
    rng = np.random.default_rng(2024)
    G_, target = 8, (1 << 24) + 5
    lens = rng.integers(1024, 3073, 9000)
    lens[100:140] = rng.choice([0, 1, 2, 5], 40)
    lens = lens[: int(np.searchsorted(np.cumsum(lens), target)) + 1]
    lens[-1] -= int(lens.sum()) - target
    lens = np.concatenate([lens, np.zeros((-len(lens)) % G_, np.int64)])       # empty sequences fill the last group
    n_seq, n_tok = len(lens), int(lens.sum())
    assert n_tok == target and lens.min() >= 0
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    ro = synth.rollout(9, n_seq // G_, G_, 4, rewards="bernoulli", equal_group_fraction=0.1)
    lp = rng.normal(-1.5, 0.5, n_tok).astype(np.float32)
    pk = synth.PackedRollout(cu, np.arange(n_seq), lp, (lp + rng.normal(0, 0.1, n_tok)).astype(np.float32),
                             (lp + rng.normal(0, 0.08, n_tok)).astype(np.float32), (rng.random(n_tok) < 0.75).astype(np.uint8),
                             np.zeros(n_tok, np.int64))
    N = int(pk.mask.sum())
    got = packed_gpu(ro, pk, beta=1e-3, N=N)
    check(ro, pk, got, 1e-3, N)


def test_packed_argument_errors():
    z = torch.zeros(16, device="cuda")
    zi = torch.zeros(4, dtype=torch.int32, device="cuda")
    m = torch.zeros(16, dtype=torch.uint8, device="cuda")
    call = lambda **kw: api.hilore_grpo_coeffs_packed(
        kw.get("rewards", z), kw.get("n_resp", 8), kw.get("G", 4), kw.get("off", 0), kw.get("n_seq", 3), kw.get("cu", zi),
        kw.get("n_tok", 16), z, z, kw.get("ref", None), m, kw.get("N", 5), None, 0.2, kw.get("beta", 0.0), 1e-6,
        kw.get("adv", z), z, None, None, check=False)
    assert call() == api.OK
    assert call(adv=None) == api.INVALID_ARG
    assert call(cu=None) == api.INVALID_ARG
    assert call(N=0) == api.ZERO_NORM
    assert call(beta=0.1) == api.INVALID_ARG
    assert call(off=6) == api.SHAPE
    assert call(n_resp=7) == api.SHAPE
    assert call(n_tok=1 << 31) == api.SHAPE
    assert call(n_seq=0, n_tok=0) == api.OK


@pytest.mark.parametrize("row_shift", [0, 1])
@pytest.mark.parametrize("min_prompt", [0, 1])
def test_packed_exposure_matches_oracle(row_shift, min_prompt):
    ro = synth.rollout(33, 6, 4, 300, lengths="uniform", min_len=1)
    pk = synth.pack_rollout(ro, 8, max_prompt=40, min_prompt=min_prompt)
    n_tok, n_seq, U = pk.n_tok, len(pk.rows), 11
    rng = np.random.default_rng(3)
    omega = (rng.standard_normal(n_tok).astype(np.float32) * 1e-4 * pk.mask).astype(np.float32)
    ld = n_tok + 5
    rms = rng.random((U, ld), dtype=np.float32) + np.float32(0.1)
    nws = api.hilore_workspace_bytes(U, n_tok)
    ws, E, sw = G.Guarded(nws), G.Guarded(U * 4), G.Guarded(4)
    api.hilore_unit_exposure_packed(G.dev(omega), G.dev(pk.mask), n_tok, dev_i32(pk.cu_seqlens), n_seq, G.dev(rms), U, ld,
                                    row_shift, 1e-8, E.ptr(), sw.ptr(), ws.ptr(), nws)
    ws.numpy(np.uint8, (nws,))
    oE, osw = oracle.unit_exposure_packed(omega, pk.mask, pk.cu_seqlens, rms, row_shift=row_shift)
    assert G.rel_err(E.numpy(np.float32, (U,)), oE).max() <= RTOL
    assert abs(float(sw.numpy(np.float32, (1,))[0]) - osw) <= RTOL * osw
