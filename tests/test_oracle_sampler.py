"""Pins for the oracle's Philox block and keep-index sampler (CPU only).

None of these checks asks the oracle to confirm itself: they use the published
Philox known answers, an independently written big-integer Philox, brute-force
selection by a full sort, set identities from Sec. 3.2.1 of the paper, the
paper's own mask examples, and inclusion statistics of a uniform K-subset.
"""
import itertools
import math
import os
import random

import numpy as np
import pytest

import oracle

M32 = 0xFFFFFFFF


# ---------------------------------------------------------------- Philox pins
def _philox_bigint(ctr, key, rounds=10):
    """Second implementation: products split into 16-bit limbs, Python integers."""
    def mulhilo(a, b):
        a0, a1 = a & 0xFFFF, a >> 16
        b0, b1 = b & 0xFFFF, b >> 16
        p00, p01, p10, p11 = a0 * b0, a0 * b1, a1 * b0, a1 * b1
        mid = (p00 >> 16) + (p01 & 0xFFFF) + (p10 & 0xFFFF)
        lo = ((mid & 0xFFFF) << 16) | (p00 & 0xFFFF)
        hi = p11 + (p01 >> 16) + (p10 >> 16) + (mid >> 16)
        return hi & M32, lo & M32
    c = list(ctr)
    k = list(key)
    for r in range(rounds):
        hi0, lo0 = mulhilo(0xD2511F53, c[0])
        hi1, lo1 = mulhilo(0xCD9E8D57, c[2])
        c = [hi1 ^ c[1] ^ k[0], lo1, hi0 ^ c[3] ^ k[1], lo0]
        k = [(k[0] + 0x9E3779B9) & M32, (k[1] + 0xBB67AE85) & M32]
    return c


def test_philox_known_answers(golden_dir):
    rows = 0
    with open(os.path.join(golden_dir, "philox4x32_10_kat.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            w = [int(t, 16) for t in line.split()]
            assert len(w) == 10
            got = oracle.philox4x32_10(w[0:4], w[4:6])
            assert [int(v) for v in got] == w[6:10]
            assert _philox_bigint(w[0:4], w[4:6]) == w[6:10]
            rows += 1
    assert rows == 3


def test_philox_matches_independent_implementation():
    rng = random.Random(7)
    for _ in range(20000):
        ctr = [rng.getrandbits(32) for _ in range(4)]
        key = [rng.getrandbits(32) for _ in range(2)]
        assert [int(v) for v in oracle.philox4x32_10(ctr, key)] == _philox_bigint(ctr, key)


def test_philox_each_input_word_matters():
    base_c, base_k = [1, 2, 3, 4], [5, 6]
    ref = list(oracle.philox4x32_10(base_c, base_k))
    for i in range(4):
        c = list(base_c); c[i] ^= 1
        assert list(oracle.philox4x32_10(c, base_k)) != ref
    for i in range(2):
        k = list(base_k); k[i] ^= 1
        assert list(oracle.philox4x32_10(base_c, k)) != ref


# ------------------------------------------------------------- keep-count rule
@pytest.mark.parametrize("N,r,K", [(16, 0.5, 8), (196, 0.5, 98), (196, 0.25, 49), (196, 0.75, 147),
                                   (196, 1.0, 196), (3136, 0.5, 1568), (784, 0.5, 392),
                                   (49, 0.5, 25), (66800, 0.5, 33400), (5, 0.01, 1), (3, 0.5, 2)])
def test_keep_count_random(N, r, K):
    # r = #kept / #all (Sec. 3.2.1), rounded half up and clamped to [1, N]
    assert oracle.keep_count(oracle.MASK_RANDOM, N, 1, r) == K


def test_keep_count_rejects_bad_ratio():
    for r in (0.0, -0.5, 1.5, float("nan")):
        assert oracle.keep_count(oracle.MASK_RANDOM, 4, 4, r) == -1
    assert oracle.keep_count(oracle.MASK_GRID, 4, 4, 0.3) == -1


@pytest.mark.parametrize("H,W", [(4, 4), (7, 7), (14, 14), (3, 5), (1, 6)])
def test_keep_count_grid_is_max_over_phases(H, W):
    hh, hw = (H + 1) // 2, (W + 1) // 2
    assert oracle.keep_count(oracle.MASK_GRID, H, W, 0.25) == hh * hw
    assert oracle.keep_count(oracle.MASK_GRID, H, W, 0.5) == (H * W + 1) // 2
    assert oracle.keep_count(oracle.MASK_GRID, H, W, 0.75) == H * W - (H // 2) * (W // 2)
    assert oracle.keep_count(oracle.MASK_GRID, H, W, 1.0) == H * W


# ---------------------------------------------------------- random keep sets
def _brute_keep(B, N, K, seed, step, offset, share=False):
    rows, offs = [], [0]
    for b in range(B):
        gid = 0 if share else offset + b
        scores = []
        for n in range(N):
            out = _philox_bigint([n >> 2, gid, step, 0], [seed & M32, seed >> 32])
            scores.append((out[n & 3] << 32) | n)
        kept = sorted(s & M32 for s in sorted(scores)[:K])
        rows += [b * N + n for n in kept]
        offs.append(len(rows))
    return rows, offs


@pytest.mark.parametrize("B,H,W,r,seed,step,off", [
    (2, 16, 1, 0.5, 0, 0, 0), (3, 5, 7, 0.25, 0xDEADBEEF12345678, 9, 4),
    (1, 1, 1, 0.5, 1, 1, 0), (2, 14, 14, 0.75, 3, 2 ** 32 - 1, 2 ** 32 - 2), (4, 3, 3, 1.0, 5, 0, 0)])
def test_random_keep_matches_full_sort(B, H, W, r, seed, step, off):
    N = H * W
    K = oracle.keep_count(oracle.MASK_RANDOM, H, W, r)
    rows, offs = oracle.sample_keep(oracle.MASK_RANDOM, B, H, W, r, seed, step, off)
    brows, boffs = _brute_keep(B, N, K, seed, step, off)
    assert rows.tolist() == brows
    assert offs.tolist() == boffs


def test_random_keep_set_identities():
    # keep and drop are disjoint and cover every position (Sec. 3.2.1)
    B, H, W, r = 5, 9, 11, 0.5
    N = H * W
    K = oracle.keep_count(oracle.MASK_RANDOM, H, W, r)
    rows, offs = oracle.sample_keep(oracle.MASK_RANDOM, B, H, W, r, seed=11, step=3)
    assert rows.dtype == np.int32 and offs.dtype == np.int32
    assert np.all(np.diff(rows) > 0)
    assert offs.tolist() == [b * K for b in range(B + 1)]
    for b in range(B):
        part = rows[offs[b]:offs[b + 1]]
        assert part.min() >= b * N and part.max() < (b + 1) * N
        keep = set(part.tolist())
        drop = set(range(b * N, (b + 1) * N)) - keep
        assert len(keep) == K and keep.isdisjoint(drop) and len(keep | drop) == N


def test_keep_ratio_one_keeps_everything():
    rows, offs = oracle.sample_keep(oracle.MASK_RANDOM, 3, 4, 5, 1.0, seed=9)
    assert rows.tolist() == list(range(60))
    assert offs.tolist() == [0, 20, 40, 60]


def test_masks_do_not_depend_on_batch_sharding():
    B, H, W, r = 8, 6, 6, 0.5
    N = H * W
    whole, _ = oracle.sample_keep(oracle.MASK_RANDOM, B, H, W, r, seed=21, step=4, sample_offset=0)
    lo, _ = oracle.sample_keep(oracle.MASK_RANDOM, 4, H, W, r, seed=21, step=4, sample_offset=0)
    hi, _ = oracle.sample_keep(oracle.MASK_RANDOM, 4, H, W, r, seed=21, step=4, sample_offset=4)
    assert whole.tolist() == lo.tolist() + (hi + 4 * N).tolist()


def test_masks_change_with_seed_step_and_sample():
    a, _ = oracle.sample_keep(oracle.MASK_RANDOM, 2, 8, 8, 0.5, seed=1, step=0)
    b, _ = oracle.sample_keep(oracle.MASK_RANDOM, 2, 8, 8, 0.5, seed=2, step=0)
    c, _ = oracle.sample_keep(oracle.MASK_RANDOM, 2, 8, 8, 0.5, seed=1, step=1)
    d, _ = oracle.sample_keep(oracle.MASK_RANDOM, 2, 8, 8, 0.5, seed=1 + (1 << 32), step=0)
    assert a.tolist() != b.tolist() and a.tolist() != c.tolist() and a.tolist() != d.tolist()
    assert (a[:32]).tolist() != (a[32:] - 64).tolist()      # samples differ


def test_share_mask_flag_repeats_sample_zero():
    N = 36
    rows, offs = oracle.sample_keep(oracle.MASK_RANDOM, 3, 6, 6, 0.5, seed=4, step=2, sample_offset=7,
                                    flags=oracle.FLAG_SHARE_MASK)
    one, _ = oracle.sample_keep(oracle.MASK_RANDOM, 1, 6, 6, 0.5, seed=4, step=2, sample_offset=0)
    assert rows.tolist() == one.tolist() + (one + N).tolist() + (one + 2 * N).tolist()


def test_random_mask_visits_positions_uniformly():
    # "statistically visit every spatial location with equal importance" (Sec. 4):
    # a uniform K-subset has P(n kept) = K/N and P(n, n' kept) = K(K-1)/(N(N-1)).
    H, W, r = 4, 3, 0.5
    N, K = H * W, 6
    trials_per_call, calls = 200, 100
    single = np.zeros(N)
    pair = np.zeros((N, N))
    for s in range(calls):
        rows, _ = oracle.sample_keep(oracle.MASK_RANDOM, trials_per_call, H, W, r, seed=1000 + s)
        pos = (rows % N).reshape(trials_per_call, K)
        onehot = np.zeros((trials_per_call, N))
        np.put_along_axis(onehot, pos, 1.0, axis=1)
        single += onehot.sum(0)
        pair += onehot.T @ onehot
    T = trials_per_call * calls
    p1 = K / N
    assert np.all(np.abs(single / T - p1) < 4.5 * math.sqrt(p1 * (1 - p1) / T))
    p2 = K * (K - 1) / (N * (N - 1))
    off = pair[~np.eye(N, dtype=bool)] / T
    assert np.all(np.abs(off - p2) < 4.5 * math.sqrt(p2 * (1 - p2) / T))


def test_all_subsets_reachable_on_tiny_case():
    # N=4, K=2: all 6 subsets should appear, roughly equally often
    seen = {}
    for s in range(30):
        rows, _ = oracle.sample_keep(oracle.MASK_RANDOM, 100, 2, 2, 0.5, seed=s)
        for t in (rows % 4).reshape(100, 2).tolist():
            seen[tuple(t)] = seen.get(tuple(t), 0) + 1
    assert sorted(seen) == list(itertools.combinations(range(4), 2))
    assert min(seen.values()) > 3000 / 6 * 0.8


# ------------------------------------------------------------ grid keep sets
def _read_examples(golden_dir):
    ex = {}
    with open(os.path.join(golden_dir, "grid_mask_examples.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, rest = line.split(None, 1)
            dims, keep = rest.split("keep=")
            d = dict(t.split("=") for t in dims.split())
            ex[name] = (int(d["H"]), int(d["W"]), [int(v) for v in keep.split()])
    return ex


def _grid_masks_seen(H, W, r, tries=64):
    seen = {}
    for s in range(tries):
        rows, _ = oracle.sample_keep(oracle.MASK_GRID, 1, H, W, r, seed=s)
        seen[tuple(rows.tolist())] = 1
    return sorted(seen)


def test_grid_quarter_contains_paper_example(golden_dir):
    H, W, keep = _read_examples(golden_dir)["example_even_h_odd_w"]
    masks = _grid_masks_seen(H, W, 0.25)
    assert len(masks) == 4                       # four phases of the 2x2 lattice
    assert tuple(keep) in masks
    # the four phases partition the map
    assert sorted(sum((list(m) for m in masks), [])) == list(range(H * W))


def test_grid_half_two_masks_cover_everything(golden_dir):
    ex = _read_examples(golden_dir)
    H, W, k0 = ex["checkerboard_phase0"]
    _, _, k1 = ex["checkerboard_phase1"]
    masks = _grid_masks_seen(H, W, 0.5)
    assert masks == sorted([tuple(k0), tuple(k1)])
    assert sorted(k0 + k1) == list(range(H * W))


def test_grid_three_quarter_is_complement_of_quarter():
    H, W = 6, 4
    q = _grid_masks_seen(H, W, 0.25)
    t = _grid_masks_seen(H, W, 0.75)
    comp = sorted(tuple(sorted(set(range(H * W)) - set(m))) for m in q)
    assert t == comp


def test_grid_counts_and_ragged_offsets_on_odd_map():
    # 7x7 at r=0.5: 25 or 24 kept per sample depending on the phase
    B, H, W = 64, 7, 7
    rows, offs = oracle.sample_keep(oracle.MASK_GRID, B, H, W, 0.5, seed=0)
    cnt = np.diff(offs)
    assert set(cnt.tolist()) == {24, 25}
    assert offs[-1] == len(rows) and np.all(np.diff(rows) > 0)
    for b in range(B):
        pos = rows[offs[b]:offs[b + 1]] - b * H * W
        par = ((pos // W) + (pos % W)) & 1
        assert len(set(par.tolist())) == 1
        assert len(pos) == (25 if par[0] == 0 else 24)
    # even dims: exactly r*N
    for r in (0.25, 0.5, 0.75, 1.0):
        _, o = oracle.sample_keep(oracle.MASK_GRID, 3, 14, 14, r, seed=2)
        assert np.diff(o).tolist() == [int(r * 196)] * 3


def test_grid_phase_is_fresh_per_step_and_sample():
    phases = set()
    for step in range(40):
        rows, _ = oracle.sample_keep(oracle.MASK_GRID, 1, 4, 4, 0.5, seed=0, step=step)
        phases.add(int(rows[0]))
    assert phases == {0, 1}
    rows, offs = oracle.sample_keep(oracle.MASK_GRID, 40, 4, 4, 0.5, seed=0, step=0)
    firsts = {int(rows[offs[b]] - 16 * b) for b in range(40)}
    assert firsts == {0, 1}


def test_grid_phase_is_the_stated_philox_word():
    """The phase rule: p = Philox4x32-10({0, g, step, 1}, seed)[0] mod #phases, with g the global sample id.
    Recomputed here with the independent big-integer Philox; another counter word, tag or output lane fails."""
    H, W, N = 6, 4, 24
    for seed, step, offset in [(0, 0, 0), (3, 17, 5), (0xDEADBEEF12345678, 2 ** 32 - 1, 2 ** 31), (9, 1, 2 ** 32 - 4)]:
        key = [seed & M32, seed >> 32]
        B = 4
        for r, phases in ((0.25, 4), (0.5, 2), (0.75, 4)):
            rows, offs = oracle.sample_keep(oracle.MASK_GRID, B, H, W, r, seed=seed, step=step, sample_offset=offset)
            for b in range(B):
                p = _philox_bigint([0, (offset + b) & M32, step, 1], key)[0] % phases
                if r == 0.5:
                    want = [n for n in range(N) if ((n // W + n % W) & 1) == p]
                else:
                    hit = [n for n in range(N) if ((n // W) & 1, (n % W) & 1) == (p >> 1, p & 1)]
                    want = hit if r == 0.25 else [n for n in range(N) if n not in hit]
                got = (rows[offs[b]:offs[b + 1]] - b * N).tolist()
                assert got == want, (seed, step, offset, r, b)
    # one mask for the whole call: every sample takes global sample 0's phase
    rows, offs = oracle.sample_keep(oracle.MASK_GRID, 3, H, W, 0.5, seed=5, step=2, sample_offset=7,
                                    flags=oracle.FLAG_SHARE_MASK)
    p = _philox_bigint([0, 0, 2, 1], [5, 0])[0] % 2
    for b in range(3):
        assert (rows[offs[b]:offs[b + 1]] - b * N).tolist() == [n for n in range(N) if ((n // W + n % W) & 1) == p]


def test_temporal_grid_phase_is_the_same_philox_word():
    T, Wf = 9, 2
    for seed, step, offset in [(1, 0, 0), (77, 5, 3)]:
        key = [seed & M32, seed >> 32]
        for r, period in ((0.25, 4), (0.5, 2), (0.75, 4)):
            rows, offs = oracle.sample_keep(oracle.MASK_TEMPORAL_GRID, 3, T, Wf, r, seed=seed, step=step,
                                            sample_offset=offset)
            for b in range(3):
                p = _philox_bigint([0, offset + b, step, 1], key)[0] % period
                frames = [f for f in range(T) if ((f % period == p) != (r == 0.75))]
                want = [f * Wf + q for f in frames for q in range(Wf)]
                assert (rows[offs[b]:offs[b + 1]] - b * T * Wf).tolist() == want, (seed, r, b)


def test_sampler_rejects_out_of_domain():
    with pytest.raises(ValueError):
        oracle.sample_keep(oracle.MASK_RANDOM, 1, 4, 4, 0.5, step=2 ** 32)
    with pytest.raises(ValueError):
        oracle.sample_keep(oracle.MASK_RANDOM, 2, 4, 4, 0.5, sample_offset=2 ** 32 - 1)
    with pytest.raises(ValueError):
        oracle.sample_keep(oracle.MASK_GRID, 1, 4, 4, 0.6)


# ---------------------------------------------------------------- temporal (whole-frame) masks
# Sec. 3.1 / 3.2.1: on video the kept subset can be a subset of frames.  Pins: the brute-force
# selection written out here, whole frames only, the reduction to the (already pinned) random
# mask on a map of T positions, sharding invariance, the counts.
@pytest.mark.parametrize("B,T,P,r,seed,step,off", [(3, 8, 5, 0.5, 0, 0, 0), (2, 16, 49, 0.25, 7, 3, 11),
                                                   (4, 5, 6, 0.75, 1, 9, 0), (1, 32, 196, 0.5, 2, 1, 4)])
def test_temporal_keep_matches_full_sort_over_frames(B, T, P, r, seed, step, off):
    rows, offs = oracle.sample_keep(oracle.MASK_TEMPORAL, B, T, P, r, seed, step, off)
    KT = max(1, min(T, math.floor(r * T + 0.5)))
    assert oracle.keep_count(oracle.MASK_TEMPORAL, T, P, r) == KT * P
    assert list(offs) == [b * KT * P for b in range(B + 1)]
    want = []
    for b in range(B):
        scores = sorted((_philox_bigint([f >> 2, off + b, step, 0], [seed & M32, seed >> 32])[f & 3] << 32) | f
                        for f in range(T))                        # the independent big-integer Philox above
        frames = sorted(s & M32 for s in scores[:KT])
        want += [b * T * P + f * P + q for f in frames for q in range(P)]
    assert list(rows) == want


def test_temporal_mask_is_the_random_mask_over_frames_expanded():
    B, T, P, r = 5, 12, 7, 0.5
    rows, _ = oracle.sample_keep(oracle.MASK_TEMPORAL, B, T, P, r, 3, 2, 6)
    frames, _ = oracle.sample_keep(oracle.MASK_RANDOM, B, T, 1, r, 3, 2, 6)          # ids b*T + f
    expanded = (frames[:, None].astype(np.int64) * P + np.arange(P)[None, :]).reshape(-1)
    assert np.array_equal(rows, expanded)
    # whole frames, nothing else: every kept frame contributes all of its P positions
    per_frame = np.bincount(rows // P, minlength=B * T)
    assert set(per_frame.tolist()) <= {0, P}


def test_temporal_mask_sharding_and_ratio_one():
    whole, _ = oracle.sample_keep(oracle.MASK_TEMPORAL, 6, 8, 4, 0.5, 5, 1, 0)
    a, _ = oracle.sample_keep(oracle.MASK_TEMPORAL, 2, 8, 4, 0.5, 5, 1, 0)
    b, _ = oracle.sample_keep(oracle.MASK_TEMPORAL, 4, 8, 4, 0.5, 5, 1, 2)
    assert np.array_equal(whole, np.concatenate([a, b + 2 * 8 * 4]))
    full, offs = oracle.sample_keep(oracle.MASK_TEMPORAL, 2, 8, 4, 1.0)
    assert np.array_equal(full, np.arange(2 * 8 * 4)) and list(offs) == [0, 32, 64]


# ---------------------------------------------------------------- frames on a lattice in time
def _frames_of(rows, B, T, P):
    """Per sample, the sorted list of kept frames; asserts that frames are kept whole."""
    per_frame = np.bincount(np.asarray(rows) // P, minlength=B * T).reshape(B, T)
    assert set(per_frame.flatten().tolist()) <= {0, P}
    return [np.flatnonzero(per_frame[b]).tolist() for b in range(B)]


def test_temporal_grid_half_is_even_or_odd_frames_and_contains_the_paper_example():
    # Sec. 3.2.1: X_keep can be X[:, even index on T, ...].  At r = 0.5 every sample keeps the even or the odd
    # frames; over many samples both phases occur, and together they cover every frame
    B, T, P = 64, 9, 5
    rows, offs = oracle.sample_keep(oracle.MASK_TEMPORAL_GRID, B, T, P, 0.5, 4, 2)
    frames = _frames_of(rows, B, T, P)
    even, odd = list(range(0, T, 2)), list(range(1, T, 2))
    assert all(f in (even, odd) for f in frames) and even in frames and odd in frames
    assert [int(offs[b + 1] - offs[b]) for b in range(B)] == [len(f) * P for f in frames]       # ragged: 5 or 4 frames
    assert oracle.keep_count(oracle.MASK_TEMPORAL_GRID, T, P, 0.5) == 5 * P


def test_temporal_grid_quarter_three_quarter_and_all():
    B, T, P = 48, 10, 3
    q, _ = oracle.sample_keep(oracle.MASK_TEMPORAL_GRID, B, T, P, 0.25, 9, 1)
    tq, _ = oracle.sample_keep(oracle.MASK_TEMPORAL_GRID, B, T, P, 0.75, 9, 1)
    fq, ftq = _frames_of(q, B, T, P), _frames_of(tq, B, T, P)
    for b in range(B):
        assert len({f % 4 for f in fq[b]}) == 1                                  # one residue class mod 4
        assert sorted(fq[b] + ftq[b]) == list(range(T))                          # same phase word: exact complements
    assert {fq[b][0] % 4 for b in range(B)} == {0, 1, 2, 3}                      # all four phases occur
    full, offs = oracle.sample_keep(oracle.MASK_TEMPORAL_GRID, 2, T, P, 1.0)
    assert np.array_equal(full, np.arange(2 * T * P))
    with pytest.raises(ValueError):
        oracle.sample_keep(oracle.MASK_TEMPORAL_GRID, 2, T, P, 0.3)


def test_temporal_grid_phase_matches_the_spatial_grid_phase_word_and_sharding():
    # the phase comes from the same Philox word as the spatial grid masks: on a T x 1 map the r = 0.5
    # checkerboard keeps (f + 0) mod 2 == p, i.e. the same frames
    B, T, P = 16, 8, 4
    rows, _ = oracle.sample_keep(oracle.MASK_TEMPORAL_GRID, B, T, P, 0.5, 11, 3, 5)
    grid, _ = oracle.sample_keep(oracle.MASK_GRID, B, T, 1, 0.5, 11, 3, 5)          # ids b*T + f
    expanded = (grid[:, None].astype(np.int64) * P + np.arange(P)[None, :]).reshape(-1)
    assert np.array_equal(rows, expanded)
    a, _ = oracle.sample_keep(oracle.MASK_TEMPORAL_GRID, 6, T, P, 0.5, 11, 3, 5)
    b, _ = oracle.sample_keep(oracle.MASK_TEMPORAL_GRID, 10, T, P, 0.5, 11, 3, 11)
    assert np.array_equal(rows, np.concatenate([a, b + 6 * T * P]))
