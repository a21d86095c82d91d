"""Calls issued from several host threads on several CUDA streams at once: every call keeps its state in its own
arguments (the launch-property cache is the only thing the host threads share), so the results are the bits of the
same calls issued one after another, and those of the oracle."""
import threading

import numpy as np
import pytest
import torch

import oracle
from paper_2609_33570_b200 import api, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


class Job:
    """One thread's work: compress with token RMS, recover, coefficients and exposure of its own inputs."""

    def __init__(self, seed, rows, cols, fmt):
        dev = torch.device("cuda", 0)
        gen = torch.Generator(device=dev)
        gen.manual_seed(seed)
        self.rows, self.cols, self.fmt, self.block = rows, cols, fmt, 64 if fmt else 0
        self.x = synth.activation_unit_device(gen, rows, cols, dev)
        self.ro = synth.rollout(seed, 1, 8, rows // 8)
        t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        self.rewards, self.lp, self.lo, self.mask = t(self.ro.rewards), t(self.ro.logp_new), t(self.ro.logp_old), t(self.ro.mask)
        self.nws = api.hilore_workspace_bytes(1, rows)
        self.alloc()

    def alloc(self):
        dev = self.x.device
        r, c = self.rows, self.cols
        self.codes = torch.full((r, c), 0xA5, dtype=torch.uint8, device=dev)
        self.scales = torch.full((r, c // 64), -7.0, dtype=torch.float32, device=dev)
        self.rms = torch.full((r,), -1.0, dtype=torch.float32, device=dev)
        self.out = torch.full((r, c), -3.0, dtype=torch.bfloat16, device=dev)
        self.omega = torch.zeros((8, r // 8), dtype=torch.float32, device=dev)
        self.expo = torch.zeros(1, dtype=torch.float32, device=dev)
        self.ws = torch.zeros(self.nws, dtype=torch.uint8, device=dev)

    def run(self, stream, reps=1):
        s = stream.cuda_stream
        for _ in range(reps):
            api.hilore_compress(self.x, self.rows, self.cols, self.cols, self.fmt, self.block, self.codes,
                                self.scales if self.fmt else None, self.rms, stream=s)
            api.hilore_recover(self.codes, self.scales if self.fmt else None, self.rows, self.cols, self.fmt, self.block,
                               self.out, self.cols, stream=s)
            api.hilore_grpo_coeffs(self.rewards, 8, 8, 0, 8, self.rows // 8, self.lp, self.lo, None, self.mask, self.ro.n_valid,
                                   None, 0.2, 0.0, 1e-6, None, self.omega, None, None, stream=s)
            api.hilore_unit_exposure(self.omega, self.mask, 8, self.rows // 8, self.rms, 1, self.rows, 0, 1e-8, self.expo,
                                     None, self.ws, self.nws, stream=s)

    def results(self):
        return (self.codes.cpu().numpy().tobytes(), self.scales.cpu().numpy().tobytes(), bits(self.out).tobytes(),
                self.rms.cpu().numpy().tobytes(), self.omega.cpu().numpy().tobytes(), self.expo.cpu().numpy().tobytes())


def test_host_threads_on_their_own_streams_give_the_bits_of_serial_calls():
    shapes = [(8192, 1536, api.FMT_E4M3FN_BLK), (4096, 8960, api.FMT_E4M3FN_RAW), (16384, 3584, api.FMT_INT8_BLK),
              (2048, 18944, api.FMT_E4M3FN_BLK)]
    jobs = [Job(100 + i, r, c, f) for i, (r, c, f) in enumerate(shapes)]
    main = torch.cuda.current_stream()
    for j in jobs:                                           # one after another, on one stream
        j.run(main)
    torch.cuda.synchronize()
    serial = [j.results() for j in jobs]
    # the first job against the oracle (the others are covered by the codec and coefficient tests)
    j0 = jobs[0]
    oc, osc = oracle.compress(bits(j0.x), j0.fmt, j0.block)
    assert np.array_equal(j0.codes.cpu().numpy(), oc)
    assert np.array_equal(j0.scales.cpu().numpy().view(np.uint32), osc.view(np.uint32))
    assert G.rel_err(j0.rms.cpu().numpy(), oracle.row_rms(bits(j0.x))).max() <= 1e-5
    for j in jobs:
        j.alloc()
    streams = [torch.cuda.Stream() for _ in jobs]
    errors = []

    def worker(j, s):
        try:
            torch.cuda.set_device(0)
            j.run(s, reps=20)                                # the same calls again and again while the others run
        except Exception as e:                               # noqa: BLE001 - reported by the assertion below
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(j, s)) for j, s in zip(jobs, streams)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    for j, want in zip(jobs, serial):
        assert j.results() == want
