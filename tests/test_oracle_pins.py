"""The CPU oracle against what the paper and the mathematics fix (no GPU).

Every check compares the oracle with something other than itself: a library
routine (cuRAND's host Philox generator, torch's float64 softmax, numpy's stable
sort), a closed form from the paper, an exact enumeration, or a statistical law.
"""
import ctypes
import glob
import itertools
import os

import numpy as np
import pytest
import torch
from scipy import stats

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------- helpers ----
def _f32(a):
    return torch.tensor(np.asarray(a, dtype=np.float32))


def _softmax64(logits, T=1.0):
    return torch.softmax(torch.as_tensor(np.asarray(logits), dtype=torch.float64) / T, dim=-1).numpy()


def _draw_from(prob, n, rng):
    """n iid draws from a small categorical law with numpy's generator (inverse cdf)."""
    cdf = np.cumsum(prob)
    cdf[-1] = 1.0
    return np.searchsorted(cdf, rng.random(n), side="right").astype(np.int32)


def _tile(row, B, K=1):
    """[V] or [K,V] logits -> [B,K,V] float32 tensor."""
    r = np.asarray(row, dtype=np.float32)
    if r.ndim == 1:
        r = r[None, :]
    return _f32(np.broadcast_to(r[None], (B,) + r.shape).copy())


# ------------------------------------------------------------------ Philox ----
def _curand():
    cands = ["/usr/local/cuda/lib64/libcurand.so.10", "libcurand.so.10"]
    cands += glob.glob(os.path.join(os.path.dirname(torch.__file__), "..", "nvidia", "curand", "lib", "libcurand.so*"))
    for c in cands:
        try:
            return ctypes.CDLL(c)
        except OSError:
            continue
    return None


def _curand_host_philox(lib, seed, offset, n):
    gen = ctypes.c_void_p()
    assert lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) == 0  # CURAND_RNG_PSEUDO_PHILOX4_32_10
    assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
    assert lib.curandSetGeneratorOffset(gen, ctypes.c_ulonglong(offset)) == 0
    out = np.zeros(n, dtype=np.uint32)
    assert lib.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(n)) == 0
    lib.curandDestroyGenerator(gen)
    return out


def test_philox_matches_curand_host_generator():
    """cuRAND's host Philox4_32_10 generator interleaves 65536 subsequences: its
    4-word block number i holds philox(counter = (i // 65536 [64-bit, words 0-1],
    i % 65536 [word 2], 0), key = seed).  That pins the round function, the
    multipliers, the key schedule, the round count and the key/seed split."""
    lib = _curand()
    if lib is None:
        pytest.skip("libcurand not loadable")
    for seed in (0, 0x123456789ABCDEF0, 0xFFFFFFFFFFFFFFFF):
        key = [seed & 0xFFFFFFFF, seed >> 32]
        # plain start: counters (0..1, 0, 0..65535, 0)
        out = _curand_host_philox(lib, seed, 0, 4 * 65536 * 2).reshape(-1, 4)
        for blk in list(range(0, 300)) + [65535, 65536, 65537, 131071]:
            ctr = [blk // 65536, 0, blk % 65536, 0]
            assert (oracle.philox4x32_10(ctr, key) == out[blk]).all(), (seed, blk)
        # large offset: carries through word 0 into word 1
        c0, c1 = 0xFFFFFFFE, 0x1234
        off = 4 * 65536 * ((c1 << 32) | c0) + 4 * 77
        out = _curand_host_philox(lib, seed, off, 4 * 65536 * 2 + 4 * 80).reshape(-1, 4)
        for blk, ctr in [(0, [c0, c1, 77, 0]), (1, [c0, c1, 78, 0]), (65536 - 77, [c0 + 1, c1, 0, 0]),
                         (2 * 65536 - 77, [0, c1 + 1, 0, 0]), (2 * 65536, [0, c1 + 1, 77, 0])]:
            assert (oracle.philox4x32_10(ctr, key) == out[blk]).all(), (seed, ctr)


def test_philox_every_counter_word_and_key_word_matters():
    base = oracle.philox4x32_10([1, 2, 3, 4], [5, 6])
    seen = {tuple(base)}
    for i in range(4):
        c = [1, 2, 3, 4]
        c[i] ^= 0x80000000
        seen.add(tuple(oracle.philox4x32_10(c, [5, 6])))
    seen.add(tuple(oracle.philox4x32_10([1, 2, 3, 4], [5 ^ 1, 6])))
    seen.add(tuple(oracle.philox4x32_10([1, 2, 3, 4], [5, 6 ^ 1])))
    # swapping two counter words is a different counter
    seen.add(tuple(oracle.philox4x32_10([1, 2, 4, 3], [5, 6])))
    seen.add(tuple(oracle.philox4x32_10([2, 1, 3, 4], [5, 6])))
    assert len(seen) == 9


def test_uniform_counter_layout_and_mapping():
    """u = ((r >> 9) + 0.5) / 2^23 of word `lane` of philox(((stream << 30) | j, b, pos, step), (seed lo, seed hi))."""
    seed = 0xDEADBEEF12345678
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for stream, j, b, pos, step, lane in [(0, 0, 0, 0, 0, 0), (1, 31615, 63, 31, 1000, 3), (1, 5, 2, 7, 9, 1),
                                          (0, 0, 17, 63, 0xFFFFFFFF, 0), (2, (1 << 30) - 1, 1, 1, 1, 2)]:
        r = oracle.philox4x32_10([(stream << 30) | j, b, pos, step], key)
        want = (float(r[lane] >> 9) + 0.5) / 8388608.0
        got = oracle.uniform(seed, stream, j, b, pos, step, lane)
        assert got == want
        assert 0.0 < got < 1.0
        assert float(np.float32(got)) == got  # exactly representable in binary32


def test_uniforms_are_uniform():
    us = np.array([oracle.uniform(42, 0, 0, b, b % 7, 3, 0) for b in range(40000)])
    assert stats.kstest(us, "uniform").pvalue > 1e-3
    us = np.array([oracle.uniform(42, 1, v >> 2, 5, 1, 3, v & 3) for v in range(40000)])
    assert stats.kstest(us, "uniform").pvalue > 1e-3
    assert abs(np.corrcoef(us[:-1], us[1:])[0, 1]) < 0.02


# ----------------------------------------------------------------- softmax ----
@pytest.mark.parametrize("T", [1.0, 0.7, 2.5])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_laws_match_library_softmax(T, dtype):
    g = torch.Generator().manual_seed(3)
    V = 777
    p = (torch.randn(V, generator=g) * 3).to(dtype)
    q = (torch.randn(V, generator=g) * 3 + 1.5).to(dtype)
    pi, rho, resid, alpha = oracle.row_laws(p, q, T)
    # T is handed over as a binary32 number, as in the library's C signature
    T32 = float(np.float32(T))
    want_pi = _softmax64(p.to(torch.float64).numpy(), T32)
    want_rho = _softmax64(q.to(torch.float64).numpy(), T32)
    np.testing.assert_allclose(pi, want_pi, rtol=1e-12, atol=0)
    np.testing.assert_allclose(rho, want_rho, rtol=1e-12, atol=0)
    assert abs(pi.sum() - 1) < 1e-12 and abs(rho.sum() - 1) < 1e-12
    # adding a constant to a row changes nothing (softmax shift invariance); exact shift in fp32
    if dtype == torch.float32:
        pi2, _, _, _ = oracle.row_laws((p.double() + 4.0).float(), q, T)
        np.testing.assert_allclose(pi2, want_pi, rtol=1e-6)


def test_minus_inf_logit_is_probability_zero():
    p = _f32([0.0, -np.inf, 1.0, -np.inf])
    q = _f32([-np.inf, 0.0, 0.0, 0.0])
    pi, rho, resid, alpha = oracle.row_laws(p, q, 1.0)
    assert pi[1] == 0 and pi[3] == 0 and rho[0] == 0
    np.testing.assert_allclose(pi, _softmax64([0.0, -np.inf, 1.0, -np.inf]), rtol=1e-14)


# ---------------------------------------- acceptance probability (P1), residual (P3) ----
def test_acceptance_probability_and_residual_identities():
    rng = np.random.default_rng(0)
    for V in (2, 4, 16, 300):
        for T in (1.0, 0.6):
            lp = rng.normal(0, 2, V).astype(np.float32)
            lq = (lp + rng.normal(0, 1.0, V)).astype(np.float32)
            pi, rho, resid, alpha = oracle.row_laws(_f32(lp), _f32(lq), T)
            T32 = float(np.float32(T))
            PI, RHO = _softmax64(lp, T32), _softmax64(lq, T32)
            # P1: sum_x rho(x) min{1, pi(x)/rho(x)} = sum_z min{pi, rho}
            acc = float(np.sum(RHO * np.minimum(1.0, PI / RHO)))
            assert abs(alpha - acc) < 1e-12
            assert abs(alpha - np.minimum(PI, RHO).sum()) < 1e-12
            # P3: the residual is a probability law, zero wherever pi <= rho, proportional to pi - rho elsewhere
            assert abs(resid.sum() - 1.0) < 1e-9
            assert (resid[PI <= RHO] == 0).all()
            pos = PI > RHO
            np.testing.assert_allclose(resid[pos], (PI - RHO)[pos] / (1.0 - acc), rtol=1e-9)
            # normaliser identity: sum [pi - rho]_+ = 1 - sum min
            assert abs(np.maximum(PI - RHO, 0).sum() - (1 - alpha)) < 1e-12


def test_emitted_token_law_equals_target_by_exact_enumeration_single_position():
    """Pr(commit x) = rho(x) min{1, pi/rho}(x) + (1 - alpha) resid(x) must equal pi(x) (proof of Theorem 1)."""
    rng = np.random.default_rng(1)
    for _ in range(20):
        V = 4
        lp = rng.normal(0, 1.5, V).astype(np.float32)
        lq = rng.normal(0, 1.5, V).astype(np.float32)
        pi, rho, resid, alpha = oracle.row_laws(_f32(lp), _f32(lq), 1.0)
        emitted = rho * np.minimum(1.0, pi / rho) + (1.0 - alpha) * resid
        np.testing.assert_allclose(emitted, _softmax64(lp), rtol=1e-12)


# --------------------------------------------------- the random procedure itself ----
def _run(q, p, tok, T, seed, step, row_len=None):
    r = oracle.spec_verify(q, p, tok, T, seed, step, row_len=row_len)
    assert r["status"] == 0
    return r


def test_acceptance_frequency_matches_sum_min():
    """Monte Carlo over Philox draws: accepted fraction within a binomial interval of alpha."""
    rng = np.random.default_rng(2)
    V, B = 4, 200000
    lp = np.array([0.3, -0.8, 1.1, 0.0], np.float32)
    lq = np.array([-0.2, 0.9, 0.1, 0.4], np.float32)
    PI, RHO = _softmax64(lp), _softmax64(lq)
    alpha = np.minimum(PI, RHO).sum()
    tok = _draw_from(RHO, B, rng).reshape(B, 1)
    r = _run(_tile(lq, B), _tile(lp, B), tok, 1.0, seed=11, step=5)
    frac = (r["accept_len"] == 1).mean()
    assert abs(frac - alpha) < 5 * np.sqrt(alpha * (1 - alpha) / B)
    # per draft token the accepted fraction is min{1, pi/rho}
    for x in range(V):
        sel = tok[:, 0] == x
        want = min(1.0, PI[x] / RHO[x])
        got = (r["accept_len"][sel] == 1).mean()
        assert abs(got - want) < 5 * np.sqrt(max(want * (1 - want), 1e-4) / sel.sum())


@pytest.mark.parametrize("V", [4, 16])
def test_residual_draw_frequencies_chi_square(V):
    rng = np.random.default_rng(3 + V)
    B = 300000
    lp = rng.normal(0, 1.2, V).astype(np.float32)
    lq = rng.normal(0, 1.2, V).astype(np.float32)
    PI, RHO = _softmax64(lp), _softmax64(lq)
    res = np.maximum(PI - RHO, 0)
    res /= res.sum()
    tok = _draw_from(RHO, B, rng).reshape(B, 1)
    r = _run(_tile(lq, B), _tile(lp, B), tok, 1.0, seed=99, step=1)
    rej = r["accept_len"] == 0
    Z = r["tokens"][rej, 0]
    assert rej.sum() > 10000
    assert (res[Z] > 0).all()  # never a token outside the residual's support
    support = np.nonzero(res > 0)[0]
    counts = np.array([(Z == x).sum() for x in support])
    chi = stats.chisquare(counts, res[support] * counts.sum())
    assert chi.pvalue > 1e-4, chi
    # confidence of the corrected token is the TARGET probability of it, not the residual's
    np.testing.assert_allclose(r["conf"][rej, 0], PI[Z], rtol=1e-12)


def test_single_position_emitted_token_law_chi_square():
    rng = np.random.default_rng(5)
    V, B = 4, 300000
    lp = np.array([1.0, 0.2, -0.5, 0.4], np.float32)
    lq = np.array([0.0, 0.8, 0.3, -1.0], np.float32)
    PI, RHO = _softmax64(lp), _softmax64(lq)
    tok = _draw_from(RHO, B, rng).reshape(B, 1)
    r = _run(_tile(lq, B), _tile(lp, B), tok, 1.0, seed=2024, step=0)
    counts = np.bincount(r["tokens"][:, 0], minlength=V)
    assert stats.chisquare(counts, PI * B).pvalue > 1e-4


def test_joint_law_of_a_window_V4_K2_exact_enumeration_and_chi_square():
    """Theorem 1 at V = 4, K = 2 with a prefix-dependent target for position 2.

    Exact part: from the oracle's per-position laws, Pr(x1, x2) enumerated over
    drafts and over accept/reject outcomes equals pi1(x1) * pi2(x2 | x1).
    Monte-Carlo part: running the procedure (a first speculative round over both positions, a
    second one over position 2 for the windows that rejected at position 1) reproduces it."""
    rng = np.random.default_rng(7)
    V = 4
    lp1 = rng.normal(0, 1, V).astype(np.float32)
    lq1 = rng.normal(0, 1, V).astype(np.float32)
    lp2 = rng.normal(0, 1, (V, V)).astype(np.float32)   # target logits of position 2 given token at position 1
    lq2 = rng.normal(0, 1, V).astype(np.float32)        # the draft does not see the prefix
    PI1, RHO1, RHO2 = _softmax64(lp1), _softmax64(lq1), _softmax64(lq2)
    PI2 = _softmax64(lp2)
    want = PI1[:, None] * PI2

    # exact enumeration through the oracle's laws
    pi1, rho1, res1, a1 = oracle.row_laws(_f32(lp1), _f32(lq1), 1.0)
    emit1 = rho1 * np.minimum(1, pi1 / rho1) + (1 - a1) * res1
    joint = np.zeros((V, V))
    for x1 in range(V):
        pi2, rho2, res2, a2 = oracle.row_laws(_f32(lp2[x1]), _f32(lq2), 1.0)
        emit2 = rho2 * np.minimum(1, pi2 / rho2) + (1 - a2) * res2
        joint[x1] = emit1[x1] * emit2
    np.testing.assert_allclose(joint, want, rtol=1e-12)

    # the procedure
    B = 300000
    d1 = _draw_from(RHO1, B, rng)
    d2 = _draw_from(RHO2, B, rng)
    q = np.stack([np.broadcast_to(lq1, (B, V)), np.broadcast_to(lq2, (B, V))], axis=1)
    p = np.stack([np.broadcast_to(lp1, (B, V)), lp2[d1]], axis=1)  # verification input uses the DRAFT prefix
    r = _run(_f32(q), _f32(p), np.stack([d1, d2], 1), 1.0, seed=5, step=0)
    x1 = r["tokens"][:, 0].copy()
    x2 = r["tokens"][:, 1].copy()
    a = r["accept_len"]
    assert ((a == 0) == (x2 == -1)).all()      # a rejection at position 1 discards the draft at position 2
    redo = np.nonzero(a == 0)[0]
    d2b = _draw_from(RHO2, len(redo), rng)
    r2 = _run(_tile(lq2, len(redo)), _f32(lp2[x1[redo]][:, None, :]), d2b.reshape(-1, 1), 1.0, seed=5, step=1)
    x2[redo] = r2["tokens"][:, 0]
    counts = np.zeros((V, V))
    np.add.at(counts, (x1, x2), 1)
    assert stats.chisquare(counts.ravel(), (want * B).ravel()).pvalue > 1e-4


def test_identical_laws_accept_everything():
    g = torch.Generator().manual_seed(0)
    B, K, V = 64, 8, 50
    q = torch.randn(B, K, V, generator=g)
    tok = torch.randint(0, V, (B, K), generator=g, dtype=torch.int32)
    for seed in range(5):
        r = _run(q, q.clone(), tok, 0.8, seed=seed, step=seed)
        assert (r["accept_len"] == K).all()
        assert np.isinf(r["gumbel_gap"]).all()  # the residual is never sampled
        assert (r["tokens"] == tok.numpy()).all()
        np.testing.assert_allclose(r["conf"], np.take_along_axis(_softmax64(q.numpy(), float(np.float32(0.8))), tok.numpy()[..., None].astype(np.int64), -1)[..., 0], rtol=1e-12)


def _golden_theorem2():
    rows = []
    with open(os.path.join(GOLDEN, "theorem2_expected_length.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                a, k, e = line.split()
                rows.append((float(a), int(k), float(e)))
    return rows


@pytest.mark.parametrize("alpha,K,expected", _golden_theorem2())
def test_mean_committed_length_matches_theorem_2(alpha, K, expected):
    """Two-token vocabulary with pi = (x, 1-x), rho = (1-x, x), x = 1 - alpha/2, so that
    sum min(pi, rho) = alpha at every position; committed = min(accept_len + 1, K)."""
    rng = np.random.default_rng(int(alpha * 1000) + K)
    B = 100000
    x = 1.0 - alpha / 2.0
    with np.errstate(divide="ignore"):
        lp = np.log(np.array([x, 1 - x])).astype(np.float32)
        lq = np.log(np.array([1 - x, x])).astype(np.float32)
    RHO = np.array([1 - x, x])
    tok = _draw_from(RHO, B * K, rng).reshape(B, K)
    r = _run(_tile(np.broadcast_to(lq, (K, 2)), B, K), _tile(np.broadcast_to(lp, (K, 2)), B, K), tok, 1.0, seed=31337, step=K)
    committed = np.minimum(r["accept_len"] + 1, K)
    sd = committed.std() / np.sqrt(B)
    assert abs(committed.mean() - expected) < 5 * sd + 1e-9
    assert ((r["tokens"] >= 0).sum(1) == committed).all()


def test_mean_committed_length_unequal_alphas():
    """Generalisation used for arbitrary logits: E[C] = sum_l prod_{i<l} alpha_i."""
    rng = np.random.default_rng(8)
    B, K, V = 100000, 4, 8
    lq = rng.normal(0, 1, (K, V)).astype(np.float32)
    lp = (lq + rng.normal(0, 0.8, (K, V))).astype(np.float32)
    PI, RHO = _softmax64(lp), _softmax64(lq)
    alphas = np.minimum(PI, RHO).sum(1)
    want = sum(np.prod(alphas[:l]) for l in range(K))
    tok = np.stack([_draw_from(RHO[i], B, rng) for i in range(K)], 1)
    r = _run(_tile(lq, B, K), _tile(lp, B, K), tok, 1.0, seed=77, step=3)
    committed = np.minimum(r["accept_len"] + 1, K)
    assert abs(committed.mean() - want) < 5 * committed.std() / np.sqrt(B)


def test_first_rejection_stops_the_window_and_sentinels():
    rng = np.random.default_rng(9)
    B, K, V = 2000, 6, 12
    lq = rng.normal(0, 1, (B, K, V)).astype(np.float32)
    lp = (lq + rng.normal(0, 1.5, (B, K, V))).astype(np.float32)
    tok = rng.integers(0, V, (B, K)).astype(np.int32)
    r = _run(_f32(lq), _f32(lp), tok, 1.0, seed=1, step=2)
    PI, RHO = _softmax64(lp), _softmax64(lq)
    for b in range(B):
        a = r["accept_len"][b]
        # replay the scan with the published uniforms
        for i in range(K):
            u = oracle.uniform(1, 0, 0, b, i, 2, 0)
            ok = u <= min(1.0, PI[b, i, tok[b, i]] / RHO[b, i, tok[b, i]])
            if not ok:
                assert a == i
                break
        else:
            assert a == K
        assert (r["tokens"][b, :a] == tok[b, :a]).all()
        assert (r["tokens"][b, a + 1:] == -1).all() and (r["conf"][b, a + 1:] == -1.0).all()
        if a < K:
            z = r["tokens"][b, a]
            assert PI[b, a, z] > RHO[b, a, z]
            assert abs(r["conf"][b, a] - PI[b, a, z]) < 1e-12


def test_row_len_limits_the_window():
    rng = np.random.default_rng(10)
    B, K, V = 50, 5, 9
    lq = rng.normal(0, 1, (B, K, V)).astype(np.float32)
    tok = rng.integers(0, V, (B, K)).astype(np.int32)
    row_len = rng.integers(0, K + 1, B).astype(np.int32)
    r = _run(_f32(lq), _f32(lq), tok, 1.0, seed=1, step=2, row_len=row_len)
    assert (r["accept_len"] == row_len).all()
    for b in range(B):
        assert (r["tokens"][b, row_len[b]:] == -1).all()


def test_greedy_temperature_zero_is_argmax_compare():
    rng = np.random.default_rng(12)
    B, K, V = 300, 5, 40
    lp = rng.normal(0, 1, (B, K, V)).astype(np.float32)
    lp[:, :, 7] = lp[:, :, 3]  # exact ties: the lowest index wins
    lq = rng.normal(0, 1, (B, K, V)).astype(np.float32)
    top = lp.argmax(-1)  # numpy returns the first maximum
    tok = np.where(rng.random((B, K)) < 0.7, top, rng.integers(0, V, (B, K))).astype(np.int32)
    r = _run(_f32(lq), _f32(lp), tok, 0.0, seed=1, step=2)
    PI1 = _softmax64(lp)
    for b in range(B):
        mism = np.nonzero(tok[b] != top[b])[0]
        a = mism[0] if len(mism) else K
        assert r["accept_len"][b] == a
        assert (r["tokens"][b, :a] == tok[b, :a]).all()
        if a < K:
            assert r["tokens"][b, a] == top[b, a]
        n = min(a + 1, K)
        np.testing.assert_allclose(r["conf"][b, :n], PI1[b, np.arange(n), r["tokens"][b, :n]], rtol=1e-12)
    assert np.isinf(r["gumbel_gap"]).all() and np.isinf(r["accept_margin"]).all()


def test_zero_draft_probability_conventions():
    # rho(x) = 0 < pi(x): accept.  pi(x) = rho(x) = 0: reject, and the replacement comes from the residual.
    lp = _f32([[[0.0, 0.0, -np.inf]]])
    lq = _f32([[[-np.inf, 0.0, -np.inf]]])
    for step in range(20):
        r = _run(lq, lp, np.array([[0]], np.int32), 1.0, 3, step)
        assert r["accept_len"][0] == 1 and r["tokens"][0, 0] == 0 and r["conf"][0, 0] == 0.5
        r = _run(lq, lp, np.array([[2]], np.int32), 1.0, 3, step)
        assert r["accept_len"][0] == 0 and r["tokens"][0, 0] == 0  # residual = (0.5, 0, 0)/0.5
    # forced rejection with zero residual mass (pi = rho) commits arg-max pi
    lp = _f32([[[0.0, 1.0, -np.inf]]])
    r = _run(lp, lp, np.array([[2]], np.int32), 1.0, 3, 0)
    assert r["accept_len"][0] == 0 and r["tokens"][0, 0] == 1


def test_data_errors_are_reported_per_window():
    rng = np.random.default_rng(13)
    B, K, V = 4, 3, 6
    lq = rng.normal(0, 1, (B, K, V)).astype(np.float32)
    lp = lq.copy()
    tok = rng.integers(0, V, (B, K)).astype(np.int32)
    bad = lp.copy()
    bad[1, 2, 4] = np.nan
    r = oracle.spec_verify(_f32(lq), _f32(bad), tok, 1.0, 0, 0)
    assert r["status"] == oracle.ERR_NONFINITE and r["accept_len"][1] == -1 and (r["accept_len"][[0, 2, 3]] == K).all()
    assert (r["tokens"][1] == -1).all()
    bad = lp.copy()
    bad[2, 0, :] = -np.inf
    assert oracle.spec_verify(_f32(lq), _f32(bad), tok, 1.0, 0, 0)["status"] == oracle.ERR_NONFINITE
    bad = lq.copy()
    bad[0, 1, 1] = np.inf
    assert oracle.spec_verify(_f32(bad), _f32(lp), tok, 1.0, 0, 0)["status"] == oracle.ERR_NONFINITE
    t2 = tok.copy()
    t2[3, 1] = V
    r = oracle.spec_verify(_f32(lq), _f32(lp), t2, 1.0, 0, 0)
    assert r["status"] == oracle.ERR_TOKEN_RANGE and r["accept_len"][3] == -1
    # entries past row_len are never looked at
    r = oracle.spec_verify(_f32(lq), _f32(lp), t2, 1.0, 0, 0, row_len=np.array([3, 3, 3, 1], np.int32))
    assert r["status"] == 0 and r["accept_len"][3] == 1
    assert oracle.spec_verify(_f32(lq), _f32(lp), tok, -1.0, 0, 0)["status"] == oracle.ERR_INVALID_ARG


def test_stream_depends_on_seed_step_batch_and_position():
    rng = np.random.default_rng(14)
    B, K, V = 256, 4, 16
    lq = rng.normal(0, 1, (1, K, V)).astype(np.float32)
    lp = (lq + rng.normal(0, 1.5, (1, K, V))).astype(np.float32)
    q, p = _tile(lq[0], B, K), _tile(lp[0], B, K)
    tok = np.broadcast_to(rng.integers(0, V, (1, K)), (B, K)).astype(np.int32).copy()
    base = _run(q, p, tok, 1.0, 1, 1)
    assert len(set(base["accept_len"].tolist())) > 1            # batch rows draw different numbers
    assert (_run(q, p, tok, 1.0, 1, 1)["tokens"] == base["tokens"]).all()  # replayable
    assert (_run(q, p, tok, 1.0, 1, 2)["tokens"] != base["tokens"]).any()
    assert (_run(q, p, tok, 1.0, 2, 1)["tokens"] != base["tokens"]).any()
    assert (_run(q, p, tok, 1.0, 1 << 32 | 1, 1)["tokens"] != base["tokens"]).any()  # high seed word is used


def test_bf16_logits_are_read_exactly():
    g = torch.Generator().manual_seed(1)
    B, K, V = 3, 4, 64
    q = torch.randn(B, K, V, generator=g).to(torch.bfloat16)
    p = (q.float() + 0.5 * torch.randn(B, K, V, generator=g)).to(torch.bfloat16)
    tok = torch.randint(0, V, (B, K), generator=g, dtype=torch.int32)
    a = oracle.spec_verify(q, p, tok, 1.0, 4, 4)
    b = oracle.spec_verify(q.float(), p.float(), tok, 1.0, 4, 4)
    assert (a["tokens"] == b["tokens"]).all() and (a["conf"] == b["conf"]).all()


def test_leading_dimension_padding_is_ignored():
    rng = np.random.default_rng(15)
    B, K, V, ld = 5, 3, 10, 16
    lq = rng.normal(0, 1, (B, K, ld)).astype(np.float32)
    lp = rng.normal(0, 1, (B, K, ld)).astype(np.float32)
    tok = rng.integers(0, V, (B, K)).astype(np.int32)
    a = oracle.spec_verify(_f32(lq), _f32(lp), tok, 1.0, 4, 4, V=V)
    lq2, lp2 = lq.copy(), lp.copy()
    lq2[:, :, V:] = 50.0
    lp2[:, :, V:] = np.nan
    b = oracle.spec_verify(_f32(lq2), _f32(lp2), tok, 1.0, 4, 4, V=V)
    c = oracle.spec_verify(_f32(lq[:, :, :V].copy()), _f32(lp[:, :, :V].copy()), tok, 1.0, 4, 4)
    assert a["status"] == b["status"] == c["status"] == 0
    assert (a["tokens"] == b["tokens"]).all() and (a["tokens"] == c["tokens"]).all()
    assert (a["conf"] == c["conf"]).all()


# ---------------------------------------------------------------- LowConf ----
def test_remask_select_matches_library_stable_sort():
    rng = np.random.default_rng(16)
    for B, L, k in [(3, 17, 5), (8, 256, 8), (2, 1024, 2), (4, 33, 40), (1, 1, 1), (2, 9, 0)]:
        conf = rng.random((B, L)).astype(np.float32)
        conf[rng.random((B, L)) < 0.3] = np.float32(0.25)       # many exact ties
        mask = (rng.random((B, L)) < 0.6).astype(np.uint8)
        pos, cnt = oracle.remask_select(conf, mask, k)
        for b in range(B):
            cand = np.nonzero(mask[b])[0]
            order = cand[np.argsort(conf[b, cand], kind="stable")]
            n = min(k, len(cand))
            assert cnt[b] == n
            assert (pos[b, :n] == order[:n]).all() and (pos[b, n:] == -1).all()


def test_remask_select_brute_force_all_tie_patterns():
    L, k = 5, 3
    levels = [np.float32(0.1), np.float32(0.5), np.float32(0.9)]
    for pattern in itertools.product(range(3), repeat=L):
        conf = np.array([[levels[i] for i in pattern]], np.float32)
        for mbits in (0b11111, 0b10110, 0b00001, 0):
            mask = np.array([[(mbits >> i) & 1 for i in range(L)]], np.uint8)
            pos, cnt = oracle.remask_select(conf, mask, k)
            cand = sorted((pattern[i], i) for i in range(L) if mask[0, i])
            want = [i for _, i in cand][:k]
            assert cnt[0] == len(want) and pos[0, :len(want)].tolist() == want


# ----------------------------------------------------------- draft sampling ----
# Algorithm 2, "Sample draft tokens x~ ~ rho"; Section 3.2.  The oracle draws by Gumbel-max;
# what pins it is the law it must produce (a library softmax), not its own arithmetic.
@pytest.mark.parametrize("V,T", [(4, 1.0), (16, 0.7), (11, 2.5)])
def test_draft_sample_frequencies_match_library_softmax_chi_square(V, T):
    rng = np.random.default_rng(100 + V)
    logits = rng.normal(0.0, 1.5, size=V).astype(np.float32)
    n = 60000
    # n independent draws: one position per batch row, so every draw has its own counter
    out = oracle.draft_sample(_tile(logits, n), T, seed=4242, step=3)
    assert out["status"] == 0
    counts = np.bincount(out["tokens"].ravel(), minlength=V)
    expected = _softmax64(logits, T) * n
    chi2 = ((counts - expected) ** 2 / expected).sum()
    assert chi2 < stats.chi2.ppf(0.9999, V - 1), (chi2, counts, expected)


def test_draft_sample_positions_steps_and_seeds_draw_independently():
    # uniform law over 8 ids, 64 windows of 8 positions: every change of the stream must show
    logits = _f32(np.zeros((64, 8, 8), dtype=np.float32))
    a = oracle.draft_sample(logits, 1.0, seed=1, step=0)["tokens"]
    assert len({tuple(r) for r in a}) > 60                         # batch rows differ
    assert (a[:, 0] != a[:, 1]).mean() > 0.7                       # positions differ
    assert (oracle.draft_sample(logits, 1.0, seed=1, step=1)["tokens"] != a).mean() > 0.7
    assert (oracle.draft_sample(logits, 1.0, seed=2, step=0)["tokens"] != a).mean() > 0.7
    # a slice of the batch drawn on its own, with its offset, repeats the full batch's draws
    b = oracle.draft_sample(logits[:10], 1.0, seed=1, step=0, batch_offset=20)["tokens"]
    assert (b == a[20:30]).all()
    # and the stream is not the one the verification step uses for its residual draw
    u_draft = oracle.uniform(1, 2, 0, 0, 0, 0, 0)
    assert u_draft != oracle.uniform(1, 1, 0, 0, 0, 0, 0) and u_draft != oracle.uniform(1, 0, 0, 0, 0, 0, 0)


def test_draft_sample_uses_one_uniform_per_vocabulary_id_as_documented():
    # brute force from the documented recipe: u_x = uniform(seed, stream 2, x >> 2, b, i, step, x & 3)
    rng = np.random.default_rng(5)
    B, K, V, T = 3, 2, 37, 0.8
    logits = rng.normal(0, 2, size=(B, K, V)).astype(np.float32)
    out = oracle.draft_sample(_f32(logits), T, seed=77, step=9)
    for b in range(B):
        for i in range(K):
            u = np.array([oracle.uniform(77, 2, x >> 2, b, i, 9, x & 3) for x in range(V)])
            scores = logits[b, i].astype(np.float64) / float(np.float32(T)) - np.log(-np.log(u))  # T is a binary32 argument
            assert out["tokens"][b, i] == int(np.argmax(scores))
            top2 = np.sort(scores)[-2:]
            assert abs(out["gumbel_gap"][b, i] - (top2[1] - top2[0])) < 1e-9


def test_draft_sample_shift_invariance_low_temperature_and_greedy():
    rng = np.random.default_rng(6)
    logits = rng.normal(0, 2, size=(5, 4, 50)).astype(np.float32)
    base = oracle.draft_sample(_f32(logits), 1.3, seed=3, step=1)["tokens"]
    # a common offset per row does not change a softmax law, nor the draw (the offset is exact in binary32)
    assert (oracle.draft_sample(_f32(logits + 64.0), 1.3, seed=3, step=1)["tokens"] == base).all()
    amax = logits.argmax(-1)
    assert (oracle.draft_sample(_f32(logits), 0.0, seed=3, step=1)["tokens"] == amax).all()
    assert (oracle.draft_sample(_f32(logits), 1e-4, seed=3, step=1)["tokens"] == amax).all()
    # ties at temperature 0: lowest index
    tied = np.zeros((1, 1, 9), dtype=np.float32)
    tied[0, 0, [3, 7]] = 2.0
    assert oracle.draft_sample(_f32(tied), 0.0, seed=0, step=0)["tokens"][0, 0] == 3


def test_draft_sample_zero_probability_entries_row_len_and_errors():
    logits = np.zeros((2, 3, 6), dtype=np.float32)
    logits[:, :, [0, 2, 5]] = -np.inf
    out = oracle.draft_sample(_f32(np.repeat(logits, 200, axis=0)), 1.0, seed=8, step=0)
    assert set(np.unique(out["tokens"])) == {1, 3, 4}              # -inf entries are never drawn
    rl = np.array([2, 0], dtype=np.int32)
    out = oracle.draft_sample(_f32(logits), 1.0, seed=8, step=0, row_len=rl)
    assert (out["tokens"][0, :2] >= 0).all() and (out["tokens"][0, 2:] == -1).all() and (out["tokens"][1] == -1).all()
    bad = np.zeros((3, 1, 4), dtype=np.float32)
    bad[0, 0, 1] = np.nan
    bad[1, 0, :] = -np.inf
    out = oracle.draft_sample(_f32(bad), 1.0, seed=8, step=0)
    assert out["status"] == oracle.ERR_NONFINITE
    assert out["tokens"][0, 0] == -1 and out["tokens"][1, 0] == -1 and out["tokens"][2, 0] >= 0
    bf = torch.tensor(np.random.default_rng(1).normal(0, 2, size=(4, 2, 33)).astype(np.float32)).to(torch.bfloat16)
    assert (oracle.draft_sample(bf, 0.9, 5, 5)["tokens"] == oracle.draft_sample(bf.float(), 0.9, 5, 5)["tokens"]).all()


# ------------------------------------------------- Algorithm 2 bookkeeping ----
from oracle import loop as oloop  # noqa: E402


def test_loop_window_is_the_first_unresolved_positions_in_order():
    rng = np.random.default_rng(0)
    for B, L, K in ((1, 1, 1), (3, 17, 4), (2, 64, 64), (4, 100, 8)):
        tokens = np.where(rng.random((B, L)) < 0.4, oloop.MASK, rng.integers(0, 50, (B, L))).astype(np.int32)
        tokens[0, :] = 7 if B > 1 else tokens[0]          # a fully resolved row
        win, rl, unres = oloop.next_window(tokens, K)
        for b in range(B):
            masked = np.nonzero(tokens[b] == oloop.MASK)[0]
            assert unres[b] == len(masked) and rl[b] == min(K, len(masked))
            assert (win[b, :rl[b]] == masked[:K]).all() and (win[b, rl[b]:] == -1).all()


def test_loop_verification_inputs_use_verified_prefix_and_draft_prefix():
    tokens = np.array([[5, -1, 6, -1, -1, 9]], dtype=np.int32)
    win, rl, _ = oloop.next_window(tokens, 3)
    drafts = np.array([[11, 12, 13]], dtype=np.int32)
    X = oloop.verification_inputs(tokens, win, rl, drafts)
    assert X[0, 0].tolist() == [5, -1, 6, -1, -1, 9]          # m = 0: nothing drafted yet
    assert X[0, 1].tolist() == [5, 11, 6, -1, -1, 9]          # m = 1: x~_{j_0} in place
    assert X[0, 2].tolist() == [5, 11, 6, 12, -1, 9]          # m = 2: x~_{j_0}, x~_{j_1}; j_2 itself still masked
    # the input of position j_m never holds its own draft or later ones
    for m in range(3):
        assert X[0, m, win[0, m]] == oloop.MASK


def test_loop_commit_counts_match_theorem_2_and_remask_restores_masks():
    tokens = np.full((3, 8), oloop.MASK, dtype=np.int32)
    conf = np.full((3, 8), -1.0, dtype=np.float32)
    in_step = np.zeros((3, 8), dtype=np.uint8)
    win, rl, _ = oloop.next_window(tokens, 4)
    accept = np.array([2, 4, -1], dtype=np.int32)              # reject at 2; all 4 accepted; data error
    out_tok = np.arange(12, dtype=np.int32).reshape(3, 4) + 100
    out_conf = np.linspace(0.1, 0.9, 12, dtype=np.float32).reshape(3, 4)
    committed = oloop.commit(tokens, conf, in_step, win, rl, accept, out_tok, out_conf)
    assert committed.tolist() == [3, 4, -1]                    # a + 1 with the corrected token; n when none rejected
    assert tokens[0].tolist() == [100, 101, 102, -1, -1, -1, -1, -1] and tokens[2].tolist() == [-1] * 8
    assert in_step.sum(axis=1).tolist() == [3, 4, 0]
    pos = np.array([[1, 0], [3, -1], [-1, -1]], dtype=np.int32)
    oloop.remask(tokens, conf, in_step, pos, np.array([2, 1, 0], dtype=np.int32))
    assert tokens[0, :3].tolist() == [-1, -1, 102] and tokens[1, 3] == -1 and conf[0, 0] == -1.0
    assert in_step.sum() == 0


def test_loop_toy_run_resolves_everything_and_remasks_the_lowest_confidences():
    rng = np.random.default_rng(3)
    B, L, K, k = 2, 20, 4, 3
    tokens = np.full((B, L), oloop.MASK, dtype=np.int32)
    conf = np.full((B, L), -1.0, dtype=np.float32)
    in_step = np.zeros((B, L), dtype=np.uint8)
    rounds = 0
    while (tokens == oloop.MASK).any():
        win, rl, _ = oloop.next_window(tokens, K)
        a = np.minimum(rng.integers(0, K + 1, B), rl).astype(np.int32)
        committed = oloop.commit(tokens, conf, in_step, win, rl, a, rng.integers(0, 99, (B, K)).astype(np.int32),
                                 rng.random((B, K)).astype(np.float32))
        assert (committed == np.minimum(a + 1, rl)).all()
        rounds += 1
        assert rounds < 100
    pos, cnt = oracle.remask_select(conf, in_step, k)
    for b in range(B):
        assert sorted(pos[b].tolist()) == sorted(np.argsort(conf[b], kind="stable")[:k].tolist())
    oloop.remask(tokens, conf, in_step, pos, cnt)
    assert ((tokens == oloop.MASK).sum(axis=1) == k).all()


# ------------------------------------------------ logits from hidden states ----
def test_lmhead_product_equals_exact_integer_arithmetic():
    """Small integer-valued bfloat16 inputs: every product and sum is an integer below 2^53, so the
    double-precision product must equal Python's exact integers."""
    from oracle import lmhead

    rng = np.random.default_rng(5)
    R, d, V = 5, 37, 11
    H = rng.integers(-9, 10, size=(R, d))
    W = rng.integers(-7, 8, size=(V, d))
    got = lmhead.lmhead_logits(torch.tensor(H, dtype=torch.bfloat16), torch.tensor(W, dtype=torch.bfloat16))
    want = [[sum(int(H[r, k]) * int(W[v, k]) for k in range(d)) for v in range(V)] for r in range(R)]
    assert got.shape == (R, V) and (got == np.array(want, dtype=np.float64)).all()
    # weight = rows of the identity: the logits are the hidden states themselves (operand order, no transpose slip)
    Hf = torch.randn(4, 6).to(torch.bfloat16)
    eye = torch.eye(6, dtype=torch.bfloat16)[:5]
    assert (lmhead.lmhead_logits(Hf, eye) == Hf.double().numpy()[:, :5]).all()


def test_float64_logit_storage_equals_the_float32_path_on_shared_values():
    """Logits that float32 holds exactly give the same verification whether stored as float32 or float64."""
    from paper_2605_14305_b200 import synth

    w = synth.TINY.with_(B=3, K=4, V=200)
    q, p, tok = synth.make_call(w, seed=12)
    a = oracle.spec_verify(q, p, tok, 0.9, 3, 4)
    b = oracle.spec_verify(q.double().numpy(), p.double().numpy(), tok, 0.9, 3, 4)
    for key in ("accept_len", "tokens", "conf", "accept_margin", "gumbel_gap"):
        assert (a[key] == b[key]).all(), key


def test_lmhead_spec_verify_is_the_verification_of_its_own_logits():
    from oracle import lmhead

    g = torch.Generator().manual_seed(2)
    B, K, d, V = 2, 3, 16, 50
    Hq = torch.randn((B * K, d), generator=g).to(torch.bfloat16)
    Hp = (Hq.float() + 0.3 * torch.randn((B * K, d), generator=g)).to(torch.bfloat16)
    W = (torch.randn((V, d), generator=g) * 0.5).to(torch.bfloat16)
    tok = torch.randint(0, V, (B, K), generator=g, dtype=torch.int32)
    out = lmhead.lmhead_spec_verify(Hq, Hp, W, tok, B, K, 1.0, 9, 1)
    again = oracle.spec_verify(out["draft_logits"], out["target_logits"], tok, 1.0, 9, 1)
    assert (out["tokens"] == again["tokens"]).all() and (out["conf"] == again["conf"]).all()
    # a common shift of one window's hidden states along a direction orthogonal to every weight row
    # leaves the logits, hence the result, unchanged
    Wn = W.clone()
    Wn[:, 0] = 0
    Hs = Hp.clone()
    Hs[:, 0] += 4.0
    o1 = lmhead.lmhead_spec_verify(Hq, Hp, Wn, tok, B, K, 1.0, 9, 1)
    o2 = lmhead.lmhead_spec_verify(Hq, Hs, Wn, tok, B, K, 1.0, 9, 1)
    assert (o1["tokens"] == o2["tokens"]).all() and (o1["conf"] == o2["conf"]).all()
