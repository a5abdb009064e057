"""GPU parity of the fused parameter sweep (gcaps_rta_sweep_batch) against the CPU oracle.

By definition a sweep over (timeslice, overhead) pairs is one independent analysis per pair, so
the oracle side is ``rta.analyse_sweep`` (a loop over ``rta.analyse``); the bar is bit-exact
equality of every value of every pair.
"""
import ctypes

import numpy as np
import pytest

from oracle import rta
from paper_2406_05221_b200 import binding, taskgen
from tests.helpers import ALL_MODES, BUSY, LITERAL, batch_of, random_tasksets

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    binding.load_library()


def sweep_parity(batch, policy, Ls, ovhs, what=""):
    ts = binding.DeviceTasksets.from_host(batch)
    k = len(ovhs)
    wc = torch.full((k, ts.n_tasks), binding.WCRT_INVALID, dtype=torch.int64, device="cuda")
    sc = torch.full((k, max(ts.n_tasksets, 0)), binding.SCHED_INVALID, dtype=torch.uint8, device="cuda")
    binding.rta_sweep(ts, policy, Ls, ovhs, out_wcrt=wc, out_sched=sc)
    torch.cuda.synchronize()
    w_ref, s_ref = rta.analyse_sweep(batch, policy, Ls if Ls is not None else [1] * k, ovhs)
    wc, sc = wc.cpu().numpy(), sc.cpu().numpy()
    for q in range(k):
        bad = np.nonzero(sc[q] != s_ref[q])[0]
        assert bad.size == 0, "%s pair %d: out_sched differs at tasksets %s" % (what, q, bad[:5])
        bad = np.nonzero(wc[q] != w_ref[q])[0]
        assert bad.size == 0, "%s pair %d: out_wcrt differs at tasks %s: %s vs oracle %s" % (
            what, q, bad[:5], wc[q][bad[:5]], w_ref[q][bad[:5]])
    # flags only: the same flags without a WCRT buffer
    _, sc2 = binding.rta_sweep(ts, policy, Ls, ovhs, want_wcrt=False)
    torch.cuda.synchronize()
    assert (sc2.cpu().numpy() == s_ref).all(), what
    return wc, sc


def test_rr_driver_model_grid_in_one_call():
    """Several tiles and a ragged tail of the driver-model workload, all 25 pairs at once."""
    w = taskgen.WORKLOADS["rr_model"]
    b = w.generate(11, 2997)
    Ls = [L for L in w.timeslices for _ in w.overheads]
    th = [t for _ in w.timeslices for t in w.overheads]
    assert len(Ls) == 25
    for policy in (1, 1 | BUSY):
        _, sc = sweep_parity(b, policy, Ls, th, "rr_model")
    assert sc.min() == 0


@pytest.mark.parametrize("policy", ALL_MODES)
def test_random_small_tasksets_all_modes(policy):
    rng = np.random.default_rng(policy + 5)
    sets = random_tasksets(rng, 2000, max_tasks=12, max_cores=4, wcet_hi=8)
    sets += random_tasksets(rng, 300, max_tasks=12, unique_prio=False)
    b = batch_of(sets)
    # repeated and changing L, L = 1, decreasing overheads, a single pair
    sweep_parity(b, policy, [1, 1, 3, 3, 7, 2, 2], [0, 1, 1, 0, 2, 2, 5], "random small")
    sweep_parity(b, policy, [4], [1], "one pair")


def test_gcaps_overhead_sweep_on_workloads():
    for name, count in (("pr1", 1000), ("sweep", 2500), ("large", 700), ("divergence", 3000)):
        w = taskgen.WORKLOADS[name]
        b = w.generate(3, count - 1, stream=0)
        eps = [0, 10, 50, 200, 1000]
        for policy in (0, BUSY):
            sweep_parity(b, policy, None, eps, name)
        sweep_parity(b, 1, [256, 1024, 1024, 4096], [0, 0, 50, 200], name)


def test_thirty_two_pairs_and_extreme_parameters():
    rng = np.random.default_rng(31)
    b = batch_of(random_tasksets(rng, 1500, max_tasks=40, max_cores=5, wcet_hi=9, max_gseg=4))
    Ls = [1 + (q * 37) % 90 for q in range(binding.MAX_SWEEP)]
    th = [(q * 11) % 7 for q in range(binding.MAX_SWEEP)]
    sweep_parity(b, 1, Ls, th, "32 pairs")
    sweep_parity(b, 0, None, th, "32 pairs gcaps")
    # a timeslice beyond every WCET, one beyond the 32-bit path, an overhead that forces the exact
    # 64-bit path for the whole sweep
    sweep_parity(b, 1, [1 << 20, 1 << 30, 5], [0, 3, 1], "huge L")
    sweep_parity(b, 1 | BUSY, [5, 9], [1 << 21, 2], "huge theta")
    sweep_parity(b, 0, None, [2, 1 << 22, 0], "huge eps")


def test_invalid_and_empty_inputs():
    rng = np.random.default_rng(2)
    b = batch_of(random_tasksets(rng, 400, max_tasks=10))
    b.period = b.period.copy()
    b.period[5] = 0                      # invalid period: that taskset is INVALID for every pair
    b.cseg_wcet = b.cseg_wcet.copy()
    b.cseg_wcet[-1] = -3
    wc, sc = sweep_parity(b, 1, [4, 8], [0, 1], "invalid")
    assert (sc == binding.SCHED_INVALID).sum() == 4
    empty = batch_of([])
    ts = binding.DeviceTasksets.from_host(empty)
    wc, sc = binding.rta_sweep(ts, 0, None, [1, 2])
    assert sc.shape == (2, 0)


def test_argument_errors():
    b = batch_of(random_tasksets(np.random.default_rng(1), 10))
    ts = binding.DeviceTasksets.from_host(b)
    with pytest.raises(binding.GcapsError) as e:
        binding.rta_sweep(ts, 1, [4] * 33, [0] * 33)
    assert e.value.code == binding.ERR_INVALID_ARG
    with pytest.raises(binding.GcapsError):
        binding.rta_sweep(ts, 1, [4, 0], [0, 0])          # L = 0 under RR
    with pytest.raises(binding.GcapsError):
        binding.rta_sweep(ts, 1, None, [0, 0])            # RR without timeslices
    with pytest.raises(binding.GcapsError):
        binding.rta_sweep(ts, 0, None, [0, -1])           # negative overhead
    lib = binding.load_library()
    rc = lib.gcaps_rta_sweep_batch(ctypes.byref(ts.c), ts.n_tasksets, 0, 0, None, None, None, None,
                                   None, 0, None)
    assert rc == binding.ERR_INVALID_ARG


def test_full_size_rr_driver_model_in_one_call_sampled():
    """The whole driver-model configuration (200,000 tasksets x 25 pairs) in the call that the
    benchmark's sweep mode times; the oracle checks a random sample of tasksets for every pair."""
    w = taskgen.WORKLOADS["rr_model"]
    b = w.generate(0, w.n_tasksets)
    ts = binding.DeviceTasksets.from_host(b)
    Ls = [L for L in w.timeslices for _ in w.overheads]
    th = [t for _ in w.timeslices for t in w.overheads]
    wc, sc = binding.rta_sweep(ts, 1, Ls, th)
    torch.cuda.synchronize()
    wc, sc = wc.cpu().numpy(), sc.cpu().numpy()
    rng = np.random.default_rng(23)
    sample = np.sort(rng.choice(b.n_tasksets, 400, replace=False))
    sub = b.select(sample)
    w_ref, s_ref = rta.analyse_sweep(sub, 1, Ls, th)
    pos = np.concatenate([np.arange(b.task_off[t], b.task_off[t + 1]) for t in sample])
    assert (sc[:, sample] == s_ref).all()
    assert (wc[:, pos] == w_ref).all()
    # any size: flags are 0/1, a converged bound never exceeds its deadline, and under round robin
    # a larger context-switch overhead never makes a taskset schedulable
    assert sc.max() <= 1
    ok = wc >= 0
    assert (wc[ok] <= np.broadcast_to(b.deadline, wc.shape)[ok]).all()
    n_th = len(w.overheads)
    for i in range(len(w.timeslices)):
        for j in range(n_th - 1):
            assert (sc[i * n_th + j] >= sc[i * n_th + j + 1]).all()
