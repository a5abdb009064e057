"""Oracle of the integer-only taskset generator -- TEST INFRASTRUCTURE ONLY.

The generation procedure is the one of the paper's Sec. 7.1 / Table 3 (tasks per CPU, the
utilisation of a CPU split over its tasks, period, number of GPU segments, segment parameters,
rate-monotonic priorities, optional worst-fit-decreasing allocation), stated here in integer
arithmetic only so that a host build and a device build can be compared bit for bit: ranges in
fixed point with 32 fractional bits, uniform spacings for the utilisation split, a log-uniform
period as round(2^y) with 2^frac a product of the constants 2^(2^-i) held with 62 fractional
bits, SplitMix64 (its published constants) keyed by (seed, stream, index) as a counter-based
random source.  Everything below is plain Python integers, one taskset at a time, slow and
obvious; it shares no code with the library (neither the C header the host and device builds
compile nor the Python package) and is imported only by the tests.

`reference_taskset(p, index)` takes any object with the integer fields of the generator's
parameter block (seed, stream, cores_lo/hi, tpc_lo/hi, util_lo/hi, log2_lo/hi, log2_hi0,
period_lo/hi, harmonic, gpu_frac, ratio_lo/hi, gpu_mode, seg_lo/hi, wfd) and returns the tasks of
taskset `index` as dicts (T, prio, core, cseg, gseg).

Pins (tests/test_igen.py): exp2_q32 against the real power of two, the procedure's ranges, sums
and distributions, rate-monotonic order, worst-fit balance, exchangeable utilisation shares.
"""
from math import isqrt

M64 = (1 << 64) - 1
GOLD = 0x9E3779B97F4A7C15


def mix64(z):
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    return z ^ (z >> 31)


class Rng:
    def __init__(self, seed, stream, index):
        k = mix64((seed + GOLD) & M64)
        k = mix64(k ^ ((stream * 0xD1B54A32D192ED03 + 0x632BE59BD9B4E019) & M64))
        k = mix64(k ^ ((index * GOLD + 0x2545F4914F6CDD1D) & M64))
        self.key, self.ctr = k, 0

    def u64(self):
        self.ctr += 1
        return mix64((self.key + self.ctr * GOLD) & M64)

    def unit(self):
        return self.u64() >> 32

    def range(self, lo, hi):
        u = self.unit()
        return lo if hi <= lo else lo + (((hi - lo) * u) >> 32)

    def int(self, lo, hi):
        x = self.u64()
        return lo if hi <= lo else lo + x % (hi - lo + 1)


ROOTS = [None, isqrt(2 << 124)]
for _ in range(2, 25):
    ROOTS.append(isqrt(ROOTS[-1] << 62))


def exp2_q32(y):
    k, f = y >> 32, (y & 0xFFFFFFFF) >> 8
    r = 1 << 62
    for i in range(1, 25):
        if (f >> (24 - i)) & 1:
            r = (r * ROOTS[i]) >> 62
    return ((r >> (61 - k)) + 1) >> 1


def split(rng, total, parts):
    w = [(1 << 32) + rng.unit() for _ in range(parts)]
    ws, spare, used, out = sum(w), total - parts, 0, []
    for j in range(parts):
        x = spare - used if j == parts - 1 else min(spare * w[j] // ws, spare - used)
        used += x
        out.append(1 + x)
    return out


def reference_taskset(p, index):
    """One taskset by the definition of csrc/igen.h, in plain Python integers."""
    rng = Rng(p.seed, p.stream, index)
    cores = min(rng.int(p.cores_lo, p.cores_hi), 64)
    harmonic = rng.unit() < p.harmonic
    util, core = [], []
    for c in range(cores):
        m = min(rng.int(p.tpc_lo, p.tpc_hi), 256 - len(util))
        U = rng.range(p.util_lo, p.util_hi)
        cuts = sorted(rng.unit() for _ in range(max(m - 1, 0)))
        before = given = 0
        for k in range(m):
            if k == m - 1:
                u = U - given
            else:
                u = (U * (cuts[k] - before)) >> 32
                before = cuts[k]
            given += u
            util.append(u)
            core.append(c)
    n = len(util)
    T = []
    for _ in range(n):
        if harmonic:
            p0 = exp2_q32(rng.range(p.log2_lo, p.log2_hi0))
            t = p0 << rng.int(0, 10)
        else:
            t = exp2_q32(rng.range(p.log2_lo, p.log2_hi))
        T.append(min(max(t, p.period_lo), p.period_hi))
    eta = [0] * n
    if p.gpu_mode == 0:
        idx = list(range(n))
        ng = min((p.gpu_frac * n + (1 << 31)) >> 32, n)
        for k in range(ng):
            j = k + rng.u64() % (n - k)
            idx[k], idx[j] = idx[j], idx[k]
            eta[idx[k]] = rng.int(max(p.seg_lo, 1), p.seg_hi)
    else:
        eta = [rng.int(p.seg_lo, p.seg_hi) for _ in range(n)]
    E = []
    for i in range(n):
        e = min(max((util[i] * T[i] + (1 << 31)) >> 32, 1), T[i])
        h = min(eta[i], 16)
        while h > 0 and e < 2 * h + 1:
            h -= 1
        E.append(e)
        eta[i] = h
        util[i] = (e << 32) // T[i]
    prio = [n - sum(1 for k in range(n) if T[k] < T[i] or (T[k] == T[i] and k < i)) for i in range(n)]
    if p.wfd:
        load, done = [0] * cores, [False] * n
        for _ in range(n):
            pick = -1
            for i in range(n):
                if not done[i] and (pick < 0 or util[i] > util[pick]):
                    pick = i
            best = min(range(cores), key=lambda c: (load[c], c))
            done[pick], core[pick] = True, best
            load[best] += util[pick]
    tasks = []
    for i in range(n):
        rho = rng.range(p.ratio_lo, p.ratio_hi)
        G = (rho * E[i] + (1 << 31)) >> 32
        gseg = []
        if eta[i] == 0:
            G = 0
        else:
            G = min(max(G, eta[i]), E[i] - eta[i] - 1)
            gseg = [(g // 5, g - g // 5) for g in split(rng, G, eta[i])]
        cseg = split(rng, E[i] - G, eta[i] + 1)
        tasks.append(dict(T=T[i], prio=prio[i], core=core[i], cseg=cseg, gseg=gseg))
    return tasks
