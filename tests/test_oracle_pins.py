"""Pins for the CPU oracle: every oracle function is checked against something
other than itself -- published known answers, library routines, brute force in
numpy written from the definitions, closed forms and limits the paper states.
No GPU is used here."""
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_rows(T, V, seed, sigma=0.7, peaks=3, dtype=np.float32):
    rng = np.random.default_rng(seed)
    zp = rng.normal(0, 2.0, (T, V))
    for t in range(T):
        cols = rng.choice(V, size=min(peaks, V), replace=False)
        zp[t, cols] += rng.uniform(4, 8, size=cols.shape[0])
    za = zp + rng.normal(0, sigma, (T, V))
    za = np.ascontiguousarray(za.astype(dtype))
    zp = np.ascontiguousarray(zp.astype(dtype))
    q = scipy.special.softmax(za.astype(np.float64), axis=1)
    tok = np.array([rng.choice(V, p=q[t]) for t in range(T)], dtype=np.int32)
    return za, zp, tok


def _to_bf16_bits(x32):
    """Round-to-nearest-even fp32 -> bf16 bit patterns, written from the format."""
    b = x32.astype(np.float32).view(np.uint32).astype(np.uint64)
    rounded = (b + 0x7FFF + ((b >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def _bf16_bits_to_f64(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


# --------------------------------------------------------------------- RNG

def test_philox_known_answers():
    n = 0
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            w = [int(x, 16) for x in line.split()]
            out = oracle.philox4x32_10(w[0:4], w[4:6])
            assert [int(x) for x in out] == w[6:10]
            n += 1
    assert n == 3


def test_uniform_is_top_24_bits_of_word0():
    for seed, g in [(0, 0), (1, 5), (0x123456789ABCDEF0, 0xFFFFFFFF), (7, 1 << 33)]:
        w = oracle.philox4x32_10([g & 0xFFFFFFFF, g >> 32, 0, 0], [seed & 0xFFFFFFFF, seed >> 32])
        assert oracle.uniform(seed, g) == (int(w[0]) >> 8) / 16777216.0


def test_uniform_distribution():
    n = 1_000_000
    z = np.zeros(n, np.float32)
    _, u, _ = oracle.accept(z, z, 1.0, seed=42, token_offset=0)
    assert u.min() >= 0.0 and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 4 * np.sqrt(1 / 12 / n)
    assert abs(u.var() - 1 / 12) < 1e-3
    assert scipy.stats.kstest(u[:200_000].astype(np.float64), "uniform").pvalue > 1e-3
    # stream depends on (seed, global index) only: offset shifts it
    _, u2, _ = oracle.accept(z[:100], z[:100], 1.0, seed=42, token_offset=1000)
    assert np.array_equal(u2, u[1000:1100])
    _, u3, _ = oracle.accept(z[:100], z[:100], 1.0, seed=43, token_offset=0)
    assert not np.array_equal(u3, u[:100])


# ---------------------------------------------------- log-softmax and gathers

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_lse_and_gather_match_library_logsumexp(dtype):
    za, zp, tok = _rand_rows(12, 777, seed=1)
    if dtype == "bf16":
        za, zp = _to_bf16_bits(za), _to_bf16_bits(zp)
        fa, fp = _bf16_bits_to_f64(za), _bf16_bits_to_f64(zp)
    else:
        fa, fp = za.astype(np.float64), zp.astype(np.float64)
    r = oracle.lse_gather(za, zp, tok)
    assert np.allclose(r["lse_a"], scipy.special.logsumexp(fa, axis=1), rtol=0, atol=1e-12)
    assert np.allclose(r["lse_p"], scipy.special.logsumexp(fp, axis=1), rtol=0, atol=1e-12)
    rows = np.arange(12)
    assert np.allclose(r["lq64"], fa[rows, tok] - scipy.special.logsumexp(fa, axis=1), atol=1e-12)
    assert np.allclose(r["lp64"], fp[rows, tok] - scipy.special.logsumexp(fp, axis=1), atol=1e-12)
    assert np.array_equal(r["lq"], r["lq64"].astype(np.float32))
    # probabilities sum to one
    assert np.allclose(np.exp(fa - r["lse_a"][:, None]).sum(1), 1.0, atol=1e-12)


def test_lse_shift_invariance_and_mask():
    za, zp, tok = _rand_rows(6, 300, seed=2)
    r0 = oracle.lse_gather(za, zp, tok)
    # a power-of-two shift keeps fp32 logits exactly representable here
    r1 = oracle.lse_gather(za + np.float32(4.0), zp - np.float32(8.0), tok)
    assert np.allclose(r0["lq64"], r1["lq64"], atol=1e-5)
    assert np.allclose(r0["lp64"], r1["lp64"], atol=1e-5)
    mask = np.array([1, 0, 1, 1, 0, 1], np.uint8)
    rm = oracle.lse_gather(za, zp, tok, mask)
    assert np.all(rm["lq"][mask == 0] == 0) and np.all(rm["lse_a"][mask == 0] == 0)
    assert np.array_equal(rm["lq"][mask == 1], r0["lq"][mask == 1])
    bad_tok = tok.copy()
    bad_tok[2] = 300
    rb = oracle.lse_gather(za, zp, bad_tok)
    assert rb["bad"].tolist() == [0, 0, 1, 0, 0, 0] and rb["lq"][2] == 0


def test_bf16_widening_is_exact():
    bits = np.array([[0x3F80, 0xBF80, 0x0000, 0x8000, 0x4049, 0xFF80]], dtype=np.uint16)  # 1,-1,0,-0,3.140625,-inf
    r = oracle.lse_gather(bits, bits, np.array([4], np.int32))
    vals = np.array([1.0, -1.0, 0.0, -0.0, 3.140625, -np.inf])
    assert np.isclose(r["lse_a"][0], scipy.special.logsumexp(vals), atol=1e-13)
    assert np.isclose(r["lq64"][0], 3.140625 - scipy.special.logsumexp(vals), atol=1e-13)


# ------------------------------------------------------------------- top-k

def _brute_topk(row64, k):
    # stable sort on negated values: ties keep ascending index order
    order = np.argsort(-row64, kind="stable")
    return order[:k].astype(np.int32)


def test_topk_against_full_stable_sort():
    za, _, _ = _rand_rows(20, 1000, seed=3)
    zq = _to_bf16_bits(za)          # bf16 rounding creates many ties
    idx = oracle.topk(zq, 50)
    f = _bf16_bits_to_f64(zq)
    for t in range(20):
        assert np.array_equal(idx[t], _brute_topk(f[t], 50))
    idx32 = oracle.topk(za, 7)
    for t in range(20):
        assert np.array_equal(idx32[t], _brute_topk(za[t].astype(np.float64), 7))


def test_topk_crafted_tie_rows():
    V, k = 64, 8
    rows = np.zeros((6, V), np.float32)
    rows[0, :] = 1.25                                  # all equal -> 0..k-1
    rows[1, :] = np.arange(V)                          # ascending ramp -> V-1, V-2, ...
    rows[2, :] = -np.arange(V)                         # descending ramp -> 0, 1, ...
    rows[3, :] = 0.0
    rows[3, [5, 9, 40]] = 2.0                          # 3 winners then ties straddling the boundary
    rows[4, :] = -np.inf
    rows[4, [63, 0]] = [1.0, 1.0]                      # peaks at both ends, rest -inf
    rows[5, :] = 0.0
    rows[5, 10] = -0.0                                 # -0 ties with +0: index order only
    rows[5, 3] = 1.0
    idx = oracle.topk(rows, k)
    assert idx[0].tolist() == list(range(8))
    assert idx[1].tolist() == list(range(63, 55, -1))
    assert idx[2].tolist() == list(range(8))
    assert idx[3].tolist() == [5, 9, 40, 0, 1, 2, 3, 4]
    assert idx[4].tolist() == [0, 63, 1, 2, 3, 4, 5, 6]
    assert idx[5].tolist() == [3, 0, 1, 2, 4, 5, 6, 7]
    m = np.array([1, 0, 1, 1, 1, 1], np.uint8)
    assert np.all(oracle.topk(rows, k, m)[1] == -1)


# ------------------------------------------------ acceptance, Z, special cases

def _pq(za, zp):
    q = scipy.special.softmax(za.astype(np.float64), axis=1)
    p = scipy.special.softmax(zp.astype(np.float64), axis=1)
    return p, q


def test_accept_probability_range_and_saturation():
    za, zp, tok = _rand_rows(400, 200, seed=4, sigma=1.5)
    r = oracle.forward(za, zp, tok, lam=1.3, k=10, seed=9)
    a = r["a"]
    assert a.min() >= 0.0 and a.max() <= 1.0
    p, q = _pq(za, zp)
    rows = np.arange(400)
    ratio = p[rows, tok] / (1.3 * q[rows, tok])
    clear = np.abs(ratio - 1) > 1e-4
    assert np.array_equal((a == 1.0)[clear], (ratio >= 1.0)[clear])
    assert np.allclose(a, np.minimum(1.0, ratio), rtol=2e-5, atol=1e-7)
    # decision is the strict comparison with the published uniform
    assert np.array_equal(r["accept"], (r["u"] < r["a"]).astype(np.uint8))
    u_direct = np.array([oracle.uniform(9, g) for g in range(400)], np.float32)
    assert np.array_equal(u_direct, r["u"])


@pytest.mark.parametrize("lam", [0.5, 1.0, 1.5, 4.0])
def test_exact_z_brute_force_and_bounds(lam):
    za, zp, tok = _rand_rows(16, 128, seed=5, sigma=1.0)
    r = oracle.forward(za, zp, tok, lam=lam, k=8, exact=True)
    p, q = _pq(za, zp)
    z_brute = np.minimum(q, p / lam).sum(1)
    assert np.allclose(r["z_exact"], z_brute, rtol=1e-12)
    # piecewise form: sum over {p/q > lam} of q + (1/lam) sum over the rest of p  (Appendix A)
    A = (p / q) > lam
    z_piece = (q * A).sum(1) + (p * ~A).sum(1) / lam
    assert np.allclose(r["z_exact"], z_piece, rtol=1e-12)
    assert np.all(r["z_exact"] <= min(1.0, 1.0 / lam) + 1e-12)
    # Z is the expected acceptance rate: sum_x q(x) a(x)
    assert np.allclose(r["z_exact"], (q * np.minimum(1.0, p / (lam * q))).sum(1), rtol=1e-12)


def test_exact_z_monotone_with_stated_slope_and_limits():
    za, zp, tok = _rand_rows(4, 64, seed=6, sigma=1.0)
    ls = oracle.lse_gather(za, zp, tok)
    p, q = _pq(za, zp)
    lams = np.linspace(0.2, 5.0, 60)
    zs = np.stack([oracle.z_exact(za, zp, ls["lse_a"], ls["lse_p"], l) for l in lams])
    assert np.all(np.diff(zs, axis=0) <= 1e-15)
    lam, h = 1.37, 1e-6
    fd = (oracle.z_exact(za, zp, ls["lse_a"], ls["lse_p"], lam + h)
          - oracle.z_exact(za, zp, ls["lse_a"], ls["lse_p"], lam - h)) / (2 * h)
    B = (p / q) <= lam
    assert np.allclose(fd, -(p * B).sum(1) / lam ** 2, rtol=1e-5)
    assert np.allclose(oracle.z_exact(za, zp, ls["lse_a"], ls["lse_p"], 1e-9), 1.0, atol=1e-12)
    assert np.all(oracle.z_exact(za, zp, ls["lse_a"], ls["lse_p"], 1e9) < 1e-8)


def test_classical_rejection_sampling_special_case():
    za, zp, tok = _rand_rows(300, 40, seed=7, sigma=0.4)
    p, q = _pq(za, zp)
    lam = float(np.float32((p / q).max() * 1.01))
    r = oracle.forward(za, zp, tok, lam=lam, k=40, seed=3)      # k = V: exact mode
    rows = np.arange(300)
    assert np.allclose(r["a"], p[rows, tok] / (lam * q[rows, tok]), rtol=2e-5)
    assert np.allclose(r["zk"], 1.0 / lam, rtol=1e-12)
    # pre-correction weight Z * max(lam, p/q) = 1: the published weight is kappa alone
    assert np.allclose(r["w64"], r["stats"]["kappa"], rtol=1e-6)
    # post-rejection distribution equals p
    qt = np.minimum(q, p / lam) / r["zk"][:, None]
    assert np.allclose(qt, p, rtol=1e-9)


@pytest.mark.parametrize("lam", [0.5, 1.0])
def test_equal_distributions_lambda_le_one(lam):
    za, _, tok = _rand_rows(64, 100, seed=8)
    r = oracle.forward(za, za.copy(), tok, lam=lam, k=100, seed=5)
    assert r["accept"].all() and np.all(r["a"] == 1.0)
    assert np.allclose(r["zk"], 1.0, atol=1e-12)
    assert r["stats"]["kappa"] == pytest.approx(1.0, abs=1e-12)
    if lam == 1.0:
        assert np.allclose(r["w64"], 1.0, atol=1e-12)
    r2 = oracle.forward(za, za.copy(), tok, lam=lam, k=5, seed=5)
    # top-k only: w_t = Zk_t / mean(Zk) * max(lam, 1), mean exactly max(lam,1)
    assert np.mean(r2["w64"]) == pytest.approx(max(lam, 1.0), rel=1e-12)


def test_equal_distributions_lambda_gt_one():
    za, _, tok = _rand_rows(64, 100, seed=8)
    r = oracle.forward(za, za.copy(), tok, lam=2.0, k=100, seed=5)
    assert np.allclose(r["a"], 0.5) and np.allclose(r["zk"], 0.5, atol=1e-12)
    assert np.allclose(r["w64"] / r["stats"]["kappa"], 1.0, atol=1e-12)


def test_lambda_to_zero_gives_plain_importance_ratio():
    za, zp, tok = _rand_rows(50, 80, seed=9, sigma=0.8)
    p, q = _pq(za, zp)
    r = oracle.forward(za, zp, tok, lam=1e-8, k=80, seed=1)
    assert r["accept"].all()
    assert np.allclose(r["zk"], 1.0, atol=1e-6) and r["stats"]["kappa"] == pytest.approx(1.0, abs=1e-6)
    rows = np.arange(50)
    assert np.allclose(r["w64"], p[rows, tok] / q[rows, tok], rtol=1e-4)


def test_weight_is_target_over_post_rejection_probability():
    za, zp, tok = _rand_rows(40, 60, seed=10, sigma=1.2)
    p, q = _pq(za, zp)
    lam = 1.5
    r = oracle.forward(za, zp, tok, lam=lam, k=60, seed=1)
    rows = np.arange(40)
    Z = np.minimum(q, p / lam).sum(1)
    P_obrs = np.minimum(q[rows, tok], p[rows, tok] / lam) / Z
    w_def = p[rows, tok] / P_obrs
    assert np.allclose(r["w64"] / r["stats"]["kappa"], w_def, rtol=1e-5)


def test_topk_estimate_underestimates_and_converges():
    za, zp, tok = _rand_rows(24, 256, seed=11, sigma=1.0)
    lam = 1.0
    prev = np.zeros(24)
    zex = oracle.forward(za, zp, tok, lam=lam, k=256)["zk"]
    errs = []
    for k in [1, 2, 4, 8, 16, 64, 128, 255, 256]:
        r = oracle.forward(za, zp, tok, lam=lam, k=k)
        assert np.all(r["zk"] <= zex + 1e-13)
        assert np.all(r["zk"] >= prev - 1e-13)
        prev = r["zk"]
        errs.append(np.abs(r["zk"] / zex - 1).mean())
    assert errs[-1] == 0.0 and errs[-2] < 1e-3 and errs[0] > errs[4] > errs[-2]
    # union is de-duplicated: brute force on one k
    r = oracle.forward(za, zp, tok, lam=lam, k=8)
    p, q = _pq(za, zp)
    for t in range(24):
        s = set(_brute_topk(za[t].astype(np.float64), 8)) | set(_brute_topk(zp[t].astype(np.float64), 8))
        s = np.array(sorted(s))
        assert r["zk"][t] == pytest.approx(np.minimum(q[t, s], p[t, s] / lam).sum(), rel=1e-12)


def test_z_equals_expected_acceptance_rate():
    # one row pair replicated; tokens drawn from q: realised acceptance -> Z
    rng = np.random.default_rng(12)
    V, n = 50, 40000
    za1, zp1, _ = _rand_rows(1, V, seed=12, sigma=1.0)
    za = np.repeat(za1, n, 0)
    zp = np.repeat(zp1, n, 0)
    p, q = _pq(za1, zp1)
    tok = rng.choice(V, size=n, p=q[0]).astype(np.int32)
    lam = 1.2
    r = oracle.forward(za, zp, tok, lam=lam, k=V, seed=77)
    Z = np.minimum(q[0], p[0] / lam).sum()
    sd = np.sqrt(Z * (1 - Z) / n)
    assert abs(r["stats"]["alpha_hat"] - Z) < 4 * sd
    assert abs(r["stats"]["mean_accept_prob"] - Z) < 4 * sd
    assert r["stats"]["kappa"] == pytest.approx(1.0, abs=4 * sd / Z)


def test_kappa_identity_and_clip():
    za, zp, tok = _rand_rows(500, 120, seed=13, sigma=1.0)
    mask = (np.arange(500) % 5 != 0).astype(np.uint8)
    r = oracle.forward(za, zp, tok, mask, lam=1.1, k=6, seed=2)
    st = r["stats"]
    assert st["n_valid"] == int(mask.sum())
    assert st["n_accept"] == int(r["accept"][mask == 1].sum()) and r["accept"][mask == 0].sum() == 0
    assert st["kappa"] * st["z_approx_mean"] == pytest.approx(st["alpha_hat"], rel=1e-12)
    assert st["z_approx_mean"] == pytest.approx(r["zk"][mask == 1].mean(), rel=1e-12)
    assert np.all(r["w"][mask == 0] == 0)
    d = (r["lp"] - r["lq"]).astype(np.float64)
    w_manual = st["kappa"] * r["zk"] * np.maximum(1.1, np.exp(d))
    assert np.allclose(r["w64"][mask == 1], w_manual[mask == 1], rtol=1e-6)
    rc = oracle.forward(za, zp, tok, mask, lam=1.1, k=6, seed=2, c1=1.05)
    assert np.allclose(rc["w64"], np.minimum(r["w64"], 1.05), rtol=1e-12)
    assert (r["w64"] > 1.05).any()


# ------------------------------------------------------------ budget -> lambda

def _g(lam, r):
    return (np.sum(r >= lam) + np.sum(r[r < lam]) / lam) / r.shape[0]


@pytest.mark.parametrize("budget", [0.05, 0.3, 0.6, 0.9, 0.999])
def test_budget_solve_hits_the_budget(budget):
    rng = np.random.default_rng(14)
    lq = rng.normal(-3, 1, 5000).astype(np.float32)
    lp = (lq + rng.normal(0, 1.2, 5000)).astype(np.float32)
    lam = oracle.lambda_from_budget(lq, lp, budget)
    r = np.exp((lp - lq).astype(np.float64))
    assert _g(lam, r) == pytest.approx(budget, abs=1e-12)
    # strictly decreasing around the solution
    assert _g(lam * 1.01, r) < budget < _g(lam * 0.99, r)


def test_budget_one_is_min_ratio_and_monotone_and_masked():
    rng = np.random.default_rng(15)
    lq = rng.normal(-3, 1, 300).astype(np.float32)
    lp = (lq + rng.normal(0, 0.7, 300)).astype(np.float32)
    r = np.exp((lp - lq).astype(np.float64))
    assert oracle.lambda_from_budget(lq, lp, 1.0) == pytest.approx(r.min(), rel=1e-15)
    lams = [oracle.lambda_from_budget(lq, lp, b) for b in (0.9, 0.7, 0.5, 0.3, 0.1)]
    assert all(x < y for x, y in zip(lams, lams[1:]))
    mask = (np.arange(300) % 3 != 0).astype(np.uint8)
    lam_m = oracle.lambda_from_budget(lq, lp, 0.5, mask)
    assert _g(lam_m, r[mask == 1]) == pytest.approx(0.5, abs=1e-12)
    # ties everywhere: all ratios equal -> g jumps from 1 to r/lam: lambda = r / b
    lam_t = oracle.lambda_from_budget(np.zeros(10, np.float32), np.full(10, 0.5, np.float32), 0.25)
    assert lam_t == pytest.approx(np.exp(0.5) / 0.25, rel=1e-12)


def test_budget_realised_acceptance():
    za, zp, tok = _rand_rows(3000, 60, seed=16, sigma=1.0)
    r = oracle.forward(za, zp, tok, budget=0.6, k=60, seed=11)
    assert r["stats"]["mean_accept_prob"] == pytest.approx(0.6, abs=2e-6)
    sd = np.sqrt(0.6 * 0.4 / 3000)
    assert abs(r["stats"]["alpha_hat"] - 0.6) < 4 * sd


# ------------------------------------------------------------------ KL facts

def test_kl_contraction_and_monotonicity():
    za, zp, tok = _rand_rows(8, 32, seed=17, sigma=1.0)
    p, q = _pq(za, zp)
    ls = oracle.lse_gather(za, zp, tok)
    kl_pq = oracle.kl_rows(za, zp, ls["lse_a"], ls["lse_p"])
    assert np.allclose(kl_pq, (p * np.log(p / q)).sum(1), rtol=1e-10)
    prev = kl_pq.copy()
    for lam in [0.05, 0.3, 0.8, 1.0, 1.5, 3.0, 10.0]:
        z = oracle.z_exact(za, zp, ls["lse_a"], ls["lse_p"], lam)
        qt = np.minimum(q, p / lam) / z[:, None]
        kl = (p * np.log(p / qt)).sum(1)
        assert np.all(kl <= prev + 1e-12)
        prev = kl
    assert np.all(prev <= kl_pq)


# ------------------------------------------------------------------ gradients

def test_gradients_by_central_differences():
    T, V = 4, 16
    za, zp, tok = _rand_rows(T, V, seed=18, sigma=0.8)
    mask = np.array([1, 1, 0, 1], np.uint8)
    rng = np.random.default_rng(18)
    adv = rng.normal(0, 1, T).astype(np.float32)
    fwd = oracle.forward(za, zp, tok, mask, lam=0.9, k=4, seed=6)
    acc = fwd["accept"].copy()
    acc[0], acc[1] = 1, 0          # one accepted, one rejected, regardless of the draw
    lam_d, g_out = 0.7, 1.3
    N = fwd["stats"]["n_valid"]
    da, dp = oracle.grad_rows(np.arange(T), za, zp, tok, acc, fwd["w"], fwd["lse_a"], fwd["lse_p"], N,
                              mask=mask, adv=adv, grad_out=g_out, lambda_distill=lam_d)
    za64, zp64 = za.astype(np.float64), zp.astype(np.float64)
    p, q = _pq(za, zp)
    rows = np.arange(T)
    consts = dict(tokens=tok, acc=acc, weight64=fwd["w"].astype(np.float64), adv64=adv.astype(np.float64),
                  logp_ref=np.log(p[rows, tok]), logq_ref=np.log(q[rows, tok]), pfix=p,
                  lambda_distill=lam_d, mask=mask)
    h = 1e-5
    for which, grad in (("a", da), ("p", dp)):
        for t in range(T):
            for v in range(V):
                zp_p, zp_m, za_p, za_m = zp64.copy(), zp64.copy(), za64.copy(), za64.copy()
                if which == "a":
                    za_p[t, v] += h
                    za_m[t, v] -= h
                else:
                    zp_p[t, v] += h
                    zp_m[t, v] -= h
                fd = g_out * (oracle.loss(za_p, zp_p, **consts) - oracle.loss(za_m, zp_m, **consts)) / (2 * h)
                assert grad[t, v] == pytest.approx(fd, rel=1e-5, abs=1e-8), (which, t, v)
    assert np.allclose(da.sum(1), 0, atol=1e-14) and np.allclose(dp.sum(1), 0, atol=1e-14)
    assert np.all(da[2] == 0) and np.all(dp[2] == 0)     # masked row
    assert np.all(dp[1] == 0) and np.any(dp[0] != 0)     # rejected / accepted row
    da0, _ = oracle.grad_rows(np.arange(T), za, zp, tok, acc, fwd["w"], fwd["lse_a"], fwd["lse_p"], N,
                              mask=mask, adv=np.zeros(T, np.float32), lambda_distill=0.0)
    assert np.all(da0 == 0)


def test_loss_function_value_by_hand():
    # J at the evaluation point: ratios are 1, KL(p||q) from the definition
    T, V = 3, 10
    za, zp, tok = _rand_rows(T, V, seed=19)
    p, q = _pq(za, zp)
    rows = np.arange(T)
    acc = np.array([1, 0, 1], np.uint8)
    w = np.array([1.5, 2.0, 0.5])
    adv = np.array([0.3, -1.0, 2.0])
    J = oracle.loss(za.astype(np.float64), zp.astype(np.float64), tok, acc, w, adv,
                    np.log(p[rows, tok]), np.log(q[rows, tok]), p, 0.4)
    by_hand = (-(acc * w * adv).sum() - adv.sum() + 0.4 * (p * np.log(p / q)).sum()) / T
    assert J == pytest.approx(by_hand, rel=1e-12)


# ---- Algorithm 1 steps 1, 3, 4 and Eq. ppo_rollout away from the first update ----------------

def test_ppo_terms_reduce_to_the_first_update_case():
    # no reference log-probs: every ratio is 1, rho is the OBRS weight, F is 1
    lq = np.array([-1.0, -2.0, -0.5], np.float32)
    lp = np.array([-1.5, -1.0, -0.7], np.float32)
    acc = np.array([1, 0, 1], np.uint8)
    w = np.array([1.2, 0.8, 2.0], np.float32)
    adv = np.array([0.5, -1.0, 2.0], np.float32)
    t = oracle.ppo_terms(lq, lp, acc, w, adv, clip=True, eps_lo=0.2, eps_hi=0.3, c2=5.0, tis_cap=2.0)
    assert np.allclose(t["rho"], w) and np.all(t["r_theta"] == 1) and np.all(t["r_omega"] == 1) and np.all(t["F"] == 1)
    assert np.allclose(t["slope_theta"], acc * w * adv) and np.allclose(t["slope_omega"], adv)
    assert np.allclose(t["obj_theta"], acc * w * adv) and np.allclose(t["obj_omega"], adv)


def test_ppo_terms_by_hand():
    # token 0: ratio above the clip with a positive advantage -> clipped, no gradient
    # token 1: ratio below the clip with a negative advantage -> clipped, no gradient
    # token 2: ratio above the clip with a negative advantage -> the min keeps the live branch
    # token 3: inside the clip range
    r = np.array([1.5, 0.6, 1.5, 1.1])
    lp = np.log(np.array([0.3, 0.2, 0.3, 0.22])).astype(np.float32)
    logp_ref = (lp.astype(np.float64) - np.log(r)).astype(np.float32)
    lq = np.log(np.array([0.25, 0.25, 0.25, 0.25])).astype(np.float32)
    acc = np.ones(4, np.uint8)
    w = np.array([2.0, 2.0, 2.0, 2.0], np.float32)
    adv = np.array([1.0, -1.0, -1.0, 1.0], np.float32)
    t = oracle.ppo_terms(lq, lp, acc, w, adv, logp_ref=logp_ref, clip=True, eps_lo=0.2, eps_hi=0.28, c2=0.8)
    r32 = np.exp(lp.astype(np.float64) - logp_ref.astype(np.float64))
    rho = 2.0 * np.minimum(1.0 / r32, 0.8)
    assert np.allclose(t["r_theta"], r32, rtol=1e-12) and np.allclose(t["rho"], rho, rtol=1e-12)
    assert t["slope_theta"][0] == 0 and t["obj_theta"][0] == pytest.approx(rho[0] * 1.28)
    assert t["slope_theta"][1] == 0 and t["obj_theta"][1] == pytest.approx(rho[1] * -0.8)
    assert t["slope_theta"][2] == pytest.approx(rho[2] * -1.0) and t["obj_theta"][2] == pytest.approx(rho[2] * -r32[2])
    assert t["slope_theta"][3] == pytest.approx(rho[3]) and t["obj_theta"][3] == pytest.approx(rho[3] * r32[3])
    # rollout side: F = min(p_omega_ref / p_inf, cap), ratio against p_omega_ref
    logq_ref = np.log(np.array([0.2, 0.3, 0.25, 0.25])).astype(np.float32)
    logp_inf = np.log(np.array([0.05, 0.3, 0.5, 0.25])).astype(np.float32)
    t = oracle.ppo_terms(lq, lp, acc, w, adv, logq_ref=logq_ref, logp_inf=logp_inf, clip=False, tis_cap=2.0)
    F = np.minimum(np.exp(logq_ref.astype(np.float64) - logp_inf.astype(np.float64)), 2.0)
    r_om = np.exp(lq.astype(np.float64) - logq_ref.astype(np.float64))
    assert F[0] == 2.0 and np.allclose(t["F"], F) and np.allclose(t["r_omega"], r_om)
    assert np.allclose(t["slope_omega"], F * adv) and np.allclose(t["obj_omega"], F * r_om * adv)
    # a rejected token carries no policy term; a masked one nothing at all
    t = oracle.ppo_terms(lq, lp, np.array([0, 1, 1, 1], np.uint8), w, adv, mask=np.array([1, 0, 1, 1], np.uint8))
    assert t["obj_theta"][0] == 0 and t["slope_theta"][0] == 0 and np.all(t["raw"][1] == 0)


def test_general_gradients_by_central_differences():
    T, V = 5, 12
    za, zp, tok = _rand_rows(T, V, seed=28, sigma=0.8)
    rng = np.random.default_rng(28)
    adv = np.array([0.8, -0.6, 1.1, -1.2, 0.4], np.float32)
    fwd = oracle.forward(za, zp, tok, None, lam=0.9, k=4, seed=6)
    acc = np.array([1, 1, 0, 1, 1], np.uint8)
    p, q = _pq(za, zp)
    rows = np.arange(T)
    # reference log-probs that put tokens on both sides of the clip range (and none on a kink)
    ratio_t = np.array([1.35, 0.7, 1.1, 1.4, 0.95])
    ratio_o = np.array([0.9, 1.3, 0.6, 0.75, 1.05])
    logp_ref = (np.log(p[rows, tok]) - np.log(ratio_t)).astype(np.float32)
    logq_ref = (np.log(q[rows, tok]) - np.log(ratio_o)).astype(np.float32)
    logp_inf = (logq_ref + rng.normal(0, 0.5, T)).astype(np.float32)
    kw = dict(clip=True, eps_lo=0.2, eps_hi=0.25)
    terms = oracle.ppo_terms(fwd["lq"], fwd["lp"], acc, fwd["w"], adv, logp_ref=logp_ref, logq_ref=logq_ref,
                             logp_inf=logp_inf, c2=0.9, tis_cap=1.5, **kw)
    lam_d, g_out = 0.3, 0.7
    da, dp = oracle.grad_rows(rows, za, zp, tok, acc, fwd["w"], fwd["lse_a"], fwd["lse_p"], T, adv=adv,
                              grad_out=g_out, lambda_distill=lam_d, ppo=terms)
    consts = dict(tokens=tok, acc=acc, weight64=terms["rho"], adv64=adv.astype(np.float64),
                  logp_ref=logp_ref.astype(np.float64), logq_ref=logq_ref.astype(np.float64), pfix=p,
                  lambda_distill=lam_d, f_actor=terms["F"], **kw)
    za64, zp64 = za.astype(np.float64), zp.astype(np.float64)
    h = 1e-6
    for which, grad in (("a", da), ("p", dp)):
        for t in range(T):
            for v in range(V):
                zp_p, zp_m, za_p, za_m = zp64.copy(), zp64.copy(), za64.copy(), za64.copy()
                if which == "a":
                    za_p[t, v] += h
                    za_m[t, v] -= h
                else:
                    zp_p[t, v] += h
                    zp_m[t, v] -= h
                fd = g_out * (oracle.loss(za_p, zp_p, **consts) - oracle.loss(za_m, zp_m, **consts)) / (2 * h)
                assert grad[t, v] == pytest.approx(fd, rel=2e-4, abs=1e-8), (which, t, v)
    # clipped tokens: the policy gradient of token 0 (ratio 1.35, A > 0) and token 1 (0.7, A < 0) is zero,
    # token 3 (1.4, A < 0) is live; the rejected token 2 has none
    assert np.all(dp[0] == 0) and np.all(dp[1] == 0) and np.all(dp[2] == 0) and np.any(dp[3] != 0)
    # without the optional inputs the general path gives the first-update gradients
    base = oracle.ppo_terms(fwd["lq"], fwd["lp"], acc, fwd["w"], adv)
    da1, dp1 = oracle.grad_rows(rows, za, zp, tok, acc, fwd["w"], fwd["lse_a"], fwd["lse_p"], T, adv=adv, ppo=base)
    da0, dp0 = oracle.grad_rows(rows, za, zp, tok, acc, fwd["w"], fwd["lse_a"], fwd["lse_p"], T, adv=adv)
    assert np.allclose(da1, da0, rtol=1e-12, atol=0) and np.allclose(dp1, dp0, rtol=1e-12, atol=0)


# ---- Theorem 3.4 per distribution: the lambda that meets an acceptance budget ------------------

def test_row_lambda_meets_the_budget_and_is_unique():
    za, zp, _ = _rand_rows(40, 300, seed=31, sigma=1.2)
    p, q = _pq(za, zp)
    for b in (0.3, 0.6, 0.9, 0.999):
        r = oracle.row_lambda(za, zp, b)
        lam = r["lam"][:, None]
        Z = np.minimum(q, p / lam).sum(1)                      # brute force from the definition
        assert np.allclose(Z, b, rtol=1e-12, atol=0)
        # Z is strictly decreasing around the solution (a unique root): a slightly smaller lambda accepts more
        assert np.all(np.minimum(q, p / (lam * 0.999)).sum(1) > b) and np.all(np.minimum(q, p / (lam * 1.001)).sum(1) < b)
    # the budget is monotone in lambda: a tighter budget needs a larger lambda
    l3, l6, l9 = (oracle.row_lambda(za, zp, b)["lam"] for b in (0.3, 0.6, 0.9))
    assert np.all(l3 > l6) and np.all(l6 > l9)
    # budget 1: the largest lambda that still accepts everything is the smallest ratio
    assert np.allclose(oracle.row_lambda(za, zp, 1.0)["lam"], (p / q).min(1), rtol=1e-12)


def test_row_lambda_closed_forms():
    # p == q: Z(lambda) = min(1, 1/lambda), so lambda = 1 / budget
    za, _, _ = _rand_rows(5, 64, seed=32)
    assert np.allclose(oracle.row_lambda(za, za, 0.4)["lam"], 2.5, rtol=1e-12)
    # two outcomes, q = (1/2, 1/2), p = (0.9, 0.1): ratios 1.8 and 0.2
    zq = np.log(np.array([[0.5, 0.5]])).astype(np.float64)
    zpp = np.log(np.array([[0.9, 0.1]])).astype(np.float64)
    za2, zp2 = zq.astype(np.float32), zpp.astype(np.float32)
    p2, q2 = _pq(za2, zp2)
    # budget 0.7: only the low-ratio outcome is cut: 0.5 + 0.1/lambda = 0.7 -> lambda = 0.5
    assert oracle.row_lambda(za2, zp2, 0.7)["lam"][0] == pytest.approx(p2[0, 1] / (0.7 - q2[0, 0]), rel=1e-12)
    assert oracle.row_lambda(za2, zp2, 0.7)["lam"][0] == pytest.approx(0.5, rel=1e-6)
    # budget 0.25: both are cut: 1/lambda = 0.25 -> lambda = 4 (above the largest ratio: classical rejection sampling)
    assert oracle.row_lambda(za2, zp2, 0.25)["lam"][0] == pytest.approx(4.0, rel=1e-6)


def test_row_lambda_kl_before_and_after():
    za, zp, _ = _rand_rows(30, 200, seed=33, sigma=1.5)
    p, q = _pq(za, zp)
    r = oracle.row_lambda(za, zp, 0.7)
    kept = np.minimum(q, p / r["lam"][:, None])
    qt = kept / kept.sum(1, keepdims=True)
    assert np.allclose(r["kl_before"], (p * np.log(p / q)).sum(1), rtol=1e-10)
    assert np.allclose(r["kl_after"], (p * np.log(p / qt)).sum(1), rtol=1e-10)
    assert np.all(r["kl_after"] <= r["kl_before"] + 1e-12)      # Theorem 3.3: the kept distribution is closer to p
    # masked rows give zeros
    m = np.ones(30, np.uint8); m[3] = 0
    rm = oracle.row_lambda(za, zp, 0.7, mask=m)
    assert rm["lam"][3] == 0 and rm["kl_after"][3] == 0 and rm["lam"][4] == r["lam"][4]


# ------------------------------------------------- sparse actor (stored top-k of the rollout model)

def _sparse_brute(zp64, q_full, inf_idx, new_idx, lam):
    """z_lo / z_hi written from their definitions with python sets, on exact double inputs."""
    p = scipy.special.softmax(zp64)
    stored = [int(x) for x in inf_idx if x >= 0]
    lo = sum(min(q_full[x], p[x] / lam) for x in stored)
    p_min = min(q_full[x] for x in stored) if stored else 1.0
    rest = 1.0 - sum(q_full[x] for x in stored)
    unknown = sum(min(p_min, p[x] / lam) for x in set(int(x) for x in new_idx if x >= 0) - set(stored))
    return lo, lo + min(unknown, max(rest, 0.0))


def test_sparse_actor_normaliser_by_hand():
    """V = 4, rollout stored its 2 best, policy top-2 holds one token the rollout did not store."""
    q = np.array([0.5, 0.3, 0.15, 0.05])
    p = np.array([0.1, 0.2, 0.6, 0.1])
    zp = np.log(p).astype(np.float32)[None, :]
    lse_p = np.array([np.log(np.exp(zp.astype(np.float64)).sum())])
    inf_idx = np.array([[0, 1]], np.int32)
    inf_logp = np.log(q[:2]).astype(np.float32)[None, :]
    new_idx = oracle.topk(zp, 2)
    assert new_idx.tolist() == [[2, 1]]
    for lam in (1.0, 2.0):
        lo, hi = oracle.z_sparse(zp, inf_idx, inf_logp, new_idx, lse_p, lam)
        want_lo = min(0.5, 0.1 / lam) + min(0.3, 0.2 / lam)
        # token 2 is unknown to the rollout record: at most the smallest stored probability (0.3), at most
        # the mass the record leaves (0.2), at most p/lambda
        want_hi = want_lo + min(min(0.3, 0.6 / lam), 0.2)
        assert lo[0] == pytest.approx(want_lo, rel=1e-6) and hi[0] == pytest.approx(want_hi, rel=1e-6)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_sparse_actor_normaliser_brackets_the_dense_estimate(dtype):
    T, V = 24, 600
    za, zp, tok = _rand_rows(T, V, 91, sigma=1.0)
    if dtype == "bf16":
        za, zp = _to_bf16_bits(za), _to_bf16_bits(zp)
        za64, zp64 = _bf16_bits_to_f64(za), _bf16_bits_to_f64(zp)
    else:
        za64, zp64 = za.astype(np.float64), zp.astype(np.float64)
    lg = oracle.lse_gather(za, zp, tok)
    q_full = scipy.special.softmax(za64, axis=1)
    prev_lo = None
    for k in (4, 16, 64, V):
        lq, inf_idx, inf_logp = oracle.rollout_record(za, tok, k)
        # the record is what the definitions give: top-k of the actor, its log-softmax at those places
        assert np.array_equal(inf_idx, oracle.topk(za, k))
        assert np.allclose(inf_logp, np.log(np.take_along_axis(q_full, inf_idx, axis=1)), rtol=0, atol=2e-6)
        assert np.allclose(lq, np.log(q_full[np.arange(T), tok]), rtol=0, atol=2e-6)
        new_idx = oracle.topk(zp, k)
        for lam in (0.7, 1.0, 2.5):
            lo, hi = oracle.z_sparse(zp, inf_idx, inf_logp, new_idx, lg["lse_p"], lam)
            dense = oracle.z_topk(za, zp, inf_idx, new_idx, lg["lse_a"], lg["lse_p"], lam)
            exact = oracle.z_exact(za, zp, lg["lse_a"], lg["lse_p"], lam)
            for t in range(T):
                # brute force on the rounded record (the oracle sees fp32 log-probs)
                qs = q_full[t].copy()
                qs[inf_idx[t]] = np.exp(inf_logp[t].astype(np.float64))
                blo, bhi = _sparse_brute(zp64[t], qs, inf_idx[t], new_idx[t], lam)
                assert lo[t] == pytest.approx(blo, rel=1e-12) and hi[t] == pytest.approx(bhi, rel=1e-12)
            tol = 1e-6
            assert np.all(lo <= dense * (1 + tol)) and np.all(dense <= hi * (1 + tol))     # the bracket
            assert np.all(lo <= exact * (1 + tol))                                         # Z_approx <= Z survives
            if k == V:                                                                     # everything stored: the dense path
                assert np.allclose(lo, exact, rtol=1e-6) and np.allclose(hi, exact, rtol=1e-6)
        lo1, _ = oracle.z_sparse(zp, inf_idx, inf_logp, new_idx, lg["lse_p"], 1.0)
        if prev_lo is not None:
            assert np.all(lo1 >= prev_lo * (1 - 1e-6))                                     # grows with the stored list
        prev_lo = lo1


def test_sparse_forward_reduces_to_the_dense_forward_when_everything_is_stored():
    T, V, k = 40, 300, 12
    za, zp, tok = _rand_rows(T, V, 92, sigma=0.9)
    mask = (np.arange(T) % 5 != 1).astype(np.uint8)
    lq, inf_idx, inf_logp = oracle.rollout_record(za, tok, V, mask)
    dense = oracle.forward(za, zp, tok, mask, lam=1.3, k=V, seed=5, c1=3.0)
    for cap in (False, True):
        sp = oracle.forward_sparse(zp, tok, lq, inf_idx, inf_logp, mask, lam=1.3, k=k, seed=5, c1=3.0, cap=cap)
        assert np.array_equal(sp["accept"], dense["accept"]) and np.array_equal(sp["u"], dense["u"])
        assert np.allclose(sp["zk"], dense["zk"], rtol=2e-6)
        assert np.allclose(sp["w64"], dense["w64"], rtol=2e-6)
        assert sp["stats"]["kappa"] == pytest.approx(dense["stats"]["kappa"], rel=2e-6)
    # with a short record the floor reading can only lose mass, and kappa makes up for it on average
    lq, inf_idx, inf_logp = oracle.rollout_record(za, tok, k, mask)
    sp = oracle.forward_sparse(zp, tok, lq, inf_idx, inf_logp, mask, lam=1.3, k=k, seed=5)
    d2 = oracle.forward(za, zp, tok, mask, lam=1.3, k=k, seed=5)
    assert np.all(sp["zk"] <= d2["zk"] * (1 + 1e-6))
    assert sp["stats"]["kappa"] >= d2["stats"]["kappa"] * (1 - 1e-9)
    assert sp["stats"]["kappa"] * sp["stats"]["z_approx_mean"] == pytest.approx(sp["stats"]["alpha_hat"], rel=1e-12)
    b = oracle.forward_sparse(zp, tok, lq, inf_idx, inf_logp, mask, budget=0.6, k=k, seed=5)
    assert b["stats"]["mean_accept_prob"] == pytest.approx(0.6, abs=1e-6)


# ------------------------------------------------------------------ output layer (fused pass)

def test_lmhead_rows_is_the_matrix_product():
    """The oracle's logits of an output layer against numpy's matmul on the exactly widened operands
    (every bf16 x bf16 product is exact in double; numpy's summation order may differ, hence 1e-12),
    and against a hand-worked 2 x 3 case."""
    rng = np.random.default_rng(93)
    T, H, V = 7, 96, 37
    hb = _to_bf16_bits(rng.normal(0, 1, (T, H)).astype(np.float32))
    wb = _to_bf16_bits(rng.normal(0, 1, (V, H)).astype(np.float32))
    rows = np.array([6, 0, 3])
    z = oracle.lmhead_rows(rows, hb, wb)
    want = _bf16_bits_to_f64(hb)[rows] @ _bf16_bits_to_f64(wb).T
    assert z.dtype == np.float32 and z.shape == (3, V)
    assert np.array_equal(z, want.astype(np.float32)) or np.allclose(z, want, rtol=1e-7, atol=1e-12)
    h2 = _to_bf16_bits(np.array([[1.0, 2.0, -0.5], [0.25, 0.0, 4.0]], np.float32))
    w2 = _to_bf16_bits(np.array([[2.0, 1.0, 1.0], [-1.0, 0.5, 8.0]], np.float32))
    z2 = oracle.lmhead_rows(np.arange(2), h2, w2)
    assert z2.tolist() == [[3.5, -4.0], [4.5, 31.75]]
