"""The calls of one microbatch step are plain stream work: they can be captured into a CUDA graph and replayed
on new data without touching the host (no allocation, no synchronisation, gating read from device memory)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_33570_b200 import api, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu
L, H, R = api.ACT_L, api.ACT_H, api.ACT_R


@pytest.mark.parametrize("one_launch", [False, True])
def test_step_captured_in_a_cuda_graph_and_replayed_on_new_data(one_launch):
    """one_launch: the score refresh through hilore_scores_plan (a kernel and the memset of its counters) instead of
    the coefficient, exposure and decide calls."""
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(0)
    shapes = [(256, 896), (256, 1536), (256, 4864)]
    U, rows = len(shapes), 256
    ro = synth.rollout(3, 1, 4, 64)                                  # 4 responses x 64 slots = 256 token rows
    x = [torch.zeros((r, c), dtype=torch.int16, device=dev) for r, c in shapes]
    codes = [torch.zeros((r, c), dtype=torch.uint8, device=dev) for r, c in shapes]
    scales = [torch.zeros((r, c // 64), dtype=torch.float32, device=dev) for r, c in shapes]
    out = [torch.zeros((r, c), dtype=torch.int16, device=dev) for r, c in shapes]
    rms = torch.zeros((U, rows), dtype=torch.float32, device=dev)
    units = [dict(x=x[i], codes=codes[i], scales=scales[i], out=out[i], row_rms=rms[i], rows=r, cols=c,
                  fmt=api.FMT_E4M3FN_BLK, block=64) for i, (r, c) in enumerate(shapes)]
    udev, uhost = api.make_unit_table(units, dev)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    rewards, lp, lo, mask = t(ro.rewards), t(ro.logp_new), t(ro.logp_old), t(ro.mask)
    omega = torch.zeros((4, 64), dtype=torch.float32, device=dev)
    expo = torch.zeros(U, dtype=torch.float32, device=dev)
    psi = torch.zeros(U, dtype=torch.float32, device=dev)
    avail = torch.tensor([L, L, H], dtype=torch.uint8, device=dev)
    action = torch.zeros(U, dtype=torch.uint8, device=dev)
    kappa = torch.ones(U, dtype=torch.float32, device=dev)
    ebar = torch.full((U,), 0.025, dtype=torch.float32, device=dev)
    nws = api.hilore_scores_plan_workspace_bytes(U, rows)
    ws = torch.zeros(nws, dtype=torch.uint8, device=dev)

    def step(stream):
        api.hilore_plan_apply(udev, uhost, U, api.PHASE_CAPTURE, None, None, None, 0, 0, avail, action, None, None, None, stream=stream)
        if one_launch:
            api.hilore_scores_plan(rewards, 4, 4, 0, 4, 64, lp, lo, None, mask, ro.n_valid, None, 0.2, 0.0, 1e-6, rms, U, rows, 0,
                                   1e-8, omega, expo, None, udev, kappa, ebar, float("inf"), float("inf"), avail, action, psi,
                                   None, None, ws, nws, stream=stream)
        else:
            api.hilore_grpo_coeffs(rewards, 4, 4, 0, 4, 64, lp, lo, None, mask, ro.n_valid, None, 0.2, 0.0, 1e-6, None, omega,
                                   None, None, stream=stream)
            api.hilore_unit_exposure(omega, mask, 4, 64, rms, U, rows, 0, 1e-8, expo, None, ws, nws, stream=stream)
            api.hilore_plan_apply(udev, uhost, U, api.PHASE_DECIDE, expo, kappa, ebar, float("inf"), float("inf"), avail, action,
                                  psi, None, None, stream=stream)
        api.hilore_plan_apply(udev, uhost, U, api.PHASE_ENCODE, None, None, None, 0, 0, avail, action, None, None, None, stream=stream)
        api.hilore_plan_apply(udev, uhost, U, api.PHASE_RECOVER, None, None, None, 0, 0, avail, action, None, None, None, stream=stream)

    side = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(side):
        step(side)                                                    # warm-up outside the capture
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        step(side)
    for trial in range(2):                                            # new data in the same buffers, replay only
        xs = [synth.activation_unit(rng, r, c) for r, c in shapes]
        for buf, a in zip(x, xs):
            buf.copy_(torch.from_numpy(a.view(np.int16)))
        for buf in codes + out:
            buf.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert action.cpu().tolist() == [L, L, L]                     # the H candidate is encoded after forward
        for i, (a, (r, c)) in enumerate(zip(xs, shapes)):
            oc, osc = oracle.compress(a, api.FMT_E4M3FN_BLK, 64)
            assert np.array_equal(codes[i].cpu().numpy(), oc)
            assert np.array_equal(out[i].cpu().numpy().view(np.uint16), oracle.recover(oc, osc, api.FMT_E4M3FN_BLK, 64))
        o_rms = np.stack([oracle.row_rms(a) for a in xs])
        adv = oracle.group_advantages(ro.rewards, 4)
        w, _, _ = oracle.grpo_coeffs(adv, ro.logp_new, ro.logp_old, None, ro.mask, N_norm=ro.n_valid)
        oE, _ = oracle.unit_exposure(w, ro.mask, o_rms)
        assert G.rel_err(expo.cpu().numpy(), oE).max() <= 1e-5
