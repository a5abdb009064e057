"""GPU parity of the best-effort flag (GCAPS_RTA_BEST_EFFORT) against the CPU oracle: bit-exact
out_wcrt (including the BEST_EFFORT sentinel) and out_sched, through the C-ABI."""
import numpy as np
import pytest

from oracle import rta
from paper_2406_05221_b200 import binding, taskgen
from tests.helpers import ALL_MODES, BEST_EFFORT, batch_of, parse_vectors, random_tasksets
from tests.test_oracle_best_effort import _demote

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    binding.load_library()


def parity(batch, policy, L, ovh, what=""):
    ts = binding.DeviceTasksets.from_host(batch)
    wc = torch.full((ts.n_tasks,), binding.WCRT_INVALID, dtype=torch.int64, device="cuda")
    sc = torch.full((max(ts.n_tasksets, 0),), binding.SCHED_INVALID, dtype=torch.uint8, device="cuda")
    binding.rta_batch(ts, policy, L, ovh, out_wcrt=wc, out_sched=sc)
    torch.cuda.synchronize()
    w_ref, s_ref, _ = rta.analyse(batch, policy, L, ovh)
    wc, sc = wc.cpu().numpy(), sc.cpu().numpy()
    bad = np.nonzero(sc != s_ref)[0]
    assert bad.size == 0, "%s: out_sched differs at tasksets %s" % (what, bad[:5])
    bad = np.nonzero(wc != w_ref)[0]
    assert bad.size == 0, "%s: out_wcrt differs at %s: %s vs oracle %s" % (what, bad[:5], wc[bad[:5]], w_ref[bad[:5]])
    return wc, sc


def test_hand_derived_vectors():
    tasks, cases = parse_vectors("table2_best_effort_vectors.txt")
    b = batch_of([tasks])
    for c in cases:
        wc, _ = parity(b, c["policy"], c["L"], c["ovh"], c["name"])
        assert wc.tolist() == c["expect"], c["name"]


@pytest.mark.parametrize("policy", ALL_MODES)
def test_random_tasksets_with_demoted_tasks(policy):
    rng = np.random.default_rng(70 + policy)
    sets, _ = _demote(random_tasksets(rng, 3000, max_tasks=12, max_cores=4, wcet_hi=8), rng)
    sets2, _ = _demote(random_tasksets(rng, 600, max_tasks=40, max_cores=6, wcet_hi=9, unique_prio=False), rng)
    b = batch_of(sets + sets2)
    for L, ovh in ((1, 0), (3, 1), (7, 2)):
        wc, sc = parity(b, policy | BEST_EFFORT, L, ovh, "demoted")
    assert (wc == binding.WCRT_BEST_EFFORT).any() and sc.max() == 1 and sc.min() == 0


def _with_best_effort_share(batch, share, rng):
    """Marks about `share` of the tasks of every taskset as best-effort: priority <- priority - n
    for the chosen ones (<= 0), the others keep their positive rate-monotonic priorities."""
    prio = batch.priority.copy()
    n = np.diff(batch.task_off)
    size = np.repeat(n, n)
    pick = rng.random(prio.shape[0]) < share
    prio[pick] -= size[pick]
    out = batch.select(np.arange(batch.n_tasksets))
    out.priority = prio
    return out


@pytest.mark.parametrize("name,count", [("pr1", 1000), ("sweep", 3000), ("large", 1200),
                                        ("rr_model", 3000), ("divergence", 5000)])
def test_workloads_with_a_share_of_best_effort_tasks(name, count):
    """The last experiment of Sec. 7.1: a percentage of the generated tasks is designated
    best-effort.  Every size bin, both policies, both modes."""
    w = taskgen.WORKLOADS[name]
    rng = np.random.default_rng(90)
    b0 = w.generate(5, count - 7, stream=len(w.streams) // 2)
    for share in (0.2, 0.6):
        b = _with_best_effort_share(b0, share, rng)
        for policy in ([0, 0x100, 1, 0x101] if "gcaps" in w.policies else [1, 0x101]):
            _, sc = parity(b, policy | BEST_EFFORT, w.timeslice_us, w.overhead_us, "%s %.1f" % (name, share))
        assert sc.max() <= 1


def test_sweep_entry_point_with_the_flag():
    rng = np.random.default_rng(8)
    sets, _ = _demote(random_tasksets(rng, 1500, max_tasks=12, max_cores=4, wcet_hi=8), rng)
    b = batch_of(sets)
    ts = binding.DeviceTasksets.from_host(b)
    for policy in (0, 1, 0x101):
        Ls, ov = [2, 2, 5, 1 << 30], [0, 3, 1, 1 << 21]
        wc, sc = binding.rta_sweep(ts, policy | BEST_EFFORT, Ls, ov)
        torch.cuda.synchronize()
        w_ref, s_ref = rta.analyse_sweep(b, policy | BEST_EFFORT, Ls, ov)
        assert (wc.cpu().numpy() == w_ref).all() and (sc.cpu().numpy() == s_ref).all()


def test_flag_is_refused_by_the_gpu_priority_entry_point():
    b = batch_of(random_tasksets(np.random.default_rng(1), 5))
    ts = binding.DeviceTasksets.from_host(b)
    with pytest.raises(binding.GcapsError) as e:
        binding.rta_gpu_priority(ts, binding.ASSIGN | BEST_EFFORT, 0)
    assert e.value.code == binding.ERR_INVALID_ARG
