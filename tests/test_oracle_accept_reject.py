"""Pins for the oracle's accept/reject rule: greedy walk, closed-form acceptance probability and
emitted-token law of speculative sampling, integer-weight accuracy, Eq. 1 against the paper's tables."""
import math
import os

import numpy as np

import oracle

from oracle.accept_reject import FRAC_BITS, integer_weights
from paper_2608_30252_b200 import inputs


def _logits_from_probs(p):
    """bf16-exact logits whose softmax is close to p (log p rounded to bf16)."""
    return oracle.round_to_bf16(np.log(np.asarray(p, dtype=np.float64)))


def test_greedy_walk_all_accept_lengths_and_ties():
    V, gamma = 9, 4
    tl = np.zeros((1, gamma + 1, V))
    best = [3, 7, 1, 5, 2]
    for i, b in enumerate(best):
        tl[0, i, b] = 2.0
    tl[0, 2, 0] = 2.0                          # exact tie at row 2: lowest index (0) wins over 1
    best[2] = 0
    for n_expect in range(gamma + 1):
        toks = np.array([best[:gamma]])
        if n_expect < gamma:
            toks[0, n_expect] = 8              # first mismatch at n_expect
        n, out = oracle.accept_reject(tl, None, toks, np.zeros((1, gamma + 1), np.float32), 0.0)
        assert n[0] == n_expect
        assert list(out[0, :n_expect]) == best[:n_expect]
        assert out[0, n_expect] == best[n_expect]
        assert (out[0, n_expect + 1:] == -1).all()


def test_spec_exp_accuracy_and_exact_points():
    assert oracle.spec_exp(0.0) == 1.0
    assert oracle.spec_exp(-65.0) == 0.0
    for e in np.linspace(-64.0, 0.0, 4001):
        assert abs(oracle.spec_exp(float(e)) - math.exp(e)) <= 4e-16 * math.exp(e)
    # powers of two come out exactly
    ln2 = math.log(2.0)
    assert abs(oracle.spec_exp(-ln2) - 0.5) < 2e-16


def test_integer_weights_total_variation_from_fp64_softmax():
    rng = np.random.default_rng(31)
    x = oracle.bf16_bits_to_f64(inputs.normal_bf16(rng, (2000,), std=4.0))
    for temp in (1.0, 0.7, 2.5):
        I = oracle.integer_weights(x, temp)
        Z = sum(I)
        p_int = np.array([i / Z for i in I])
        z = x / float(np.float32(temp))
        p = np.exp(z - z.max()); p /= p.sum()
        assert max(I) == 1 << FRAC_BITS
        assert 0.5 * np.abs(p_int - p).sum() < len(x) * 2.0 ** -39


def test_acceptance_probability_is_one_minus_total_variation():
    """p = (.4,.3,.2,.1), q = (.1,.2,.3,.4): P(accept) = sum_x min(p,q) = 0.6; the residual is
    (.75,.25,0,0); the emitted token follows p exactly (Leviathan et al.'s losslessness)."""
    p = [0.4, 0.3, 0.2, 0.1]; q = [0.1, 0.2, 0.3, 0.4]
    tl = np.stack([_logits_from_probs(p), _logits_from_probs(p)])[None]      # gamma = 1
    dl = _logits_from_probs(q)[None, None]
    Ip = oracle.integer_weights(tl[0, 0], 1.0); Iq = oracle.integer_weights(dl[0, 0], 1.0)
    pt = np.array(Ip) / sum(Ip); qt = np.array(Iq) / sum(Iq)                 # the quantised laws
    assert np.allclose(pt, p, atol=3e-3) and np.allclose(qt, q, atol=3e-3)
    rng = np.random.default_rng(32)
    N = 60000
    xs = rng.choice(4, size=N, p=qt)
    us = inputs.uniforms_24bit(rng, (N, 2))
    acc = 0
    emitted = np.zeros(4)
    resid = np.zeros(4)
    for x, u in zip(xs, us):
        n, out = oracle.accept_reject(tl, dl, np.array([[x]]), u[None], 1.0)
        acc += int(n[0])
        emitted[out[0, 0]] += 1
        if n[0] == 0:
            resid[out[0, 0]] += 1
    p_acc = np.minimum(pt, qt).sum()
    assert abs(p_acc - 0.6) < 5e-3
    assert abs(acc / N - p_acc) < 4 * math.sqrt(p_acc * (1 - p_acc) / N)
    for j in range(4):
        assert abs(emitted[j] / N - pt[j]) < 4 * math.sqrt(pt[j] * (1 - pt[j]) / N) + 1e-9
    r = np.maximum(pt - qt, 0); r /= r.sum()
    assert np.allclose(r, [0.75, 0.25, 0, 0], atol=2e-2)
    nrej = resid.sum()
    assert resid[2] == 0 and resid[3] == 0
    assert abs(resid[0] / nrej - r[0]) < 4 * math.sqrt(r[0] * (1 - r[0]) / nrej)


def test_sampling_exact_decisions_by_enumeration():
    """Tiny case checked against the rule written with fractions: accept iff u < p(x)/q(x)."""
    from fractions import Fraction
    tl = np.array([[[0.0, -1.0, 1.0], [0.5, 0.0, -0.5]]])
    dl = np.array([[[1.0, 0.0, 0.0]]])
    Ip = oracle.integer_weights(tl[0, 0], 1.0); Iq = oracle.integer_weights(dl[0, 0], 1.0)
    Ib = oracle.integer_weights(tl[0, 1], 1.0)
    for x in range(3):
        ratio = Fraction(Ip[x] * sum(Iq), Iq[x] * sum(Ip))
        for k in (0, 1, 1 << 20, 3 << 22, (1 << 24) - 1):
            for kf in (0, 5 << 20, (1 << 24) - 1):
                u = np.array([[k * 2.0 ** -24, kf * 2.0 ** -24]], dtype=np.float32)
                n, out = oracle.accept_reject(tl, dl, np.array([[x]]), u, 1.0)
                assert (n[0] == 1) == (Fraction(k, 1 << 24) < ratio)
                if n[0] == 1:
                    w = Ib
                else:
                    w = [max(0, a * sum(Iq) - b * sum(Ip)) >> 48 for a, b in zip(Ip, Iq)]
                cdf = np.cumsum([Fraction(v, sum(w)) for v in w])
                expect = next(j for j in range(3) if Fraction((kf * sum(w)) >> 24, sum(w)) < cdf[j])
                assert out[0, n[0]] == expect


def test_identical_distributions_always_accept_and_low_temperature_is_greedy():
    rng = np.random.default_rng(33)
    tl = oracle.bf16_bits_to_f64(inputs.normal_bf16(rng, (1, 4, 50), std=3.0))
    dl = tl[:, :3].copy()
    for _ in range(20):
        toks = rng.integers(0, 50, (1, 3))
        u = inputs.uniforms_24bit(rng, (1, 4))
        n, _ = oracle.accept_reject(tl, dl, toks, u, 1.0)
        assert n[0] == 3                      # p == q: ratio 1, u < 1 always
    greedy_toks = tl[:, :3].argmax(-1)
    n_g, out_g = oracle.accept_reject(tl, None, greedy_toks, np.zeros((1, 4), np.float32), 0.0)
    one_hot = np.full((1, 3, 50), -30.0); np.put_along_axis(one_hot, greedy_toks[..., None], 0.0, -1)
    n_s, out_s = oracle.accept_reject(tl, one_hot, greedy_toks, inputs.uniforms_24bit(rng, (1, 4)), 0.01)
    assert n_g[0] == n_s[0] == 3 and np.array_equal(out_g, out_s)


def test_residual_weight_sum_fits_64_bits_below_vocab_2_pow_17():
    """The sampler's largest sum: p and q flat on disjoint halves of the vocabulary give sum R = (V/2)^2 2^32 =
    V^2 2^30 (every weight is 2^40, each residual 2^40 (V/2) 2^40 >> 48).  It reaches 2^64 exactly at V = 2^17,
    which is why a 64-bit implementation must refuse V >= 131072 when sampling; V = 131070 still fits."""
    for V, fits in ((131070, True), (131072, False)):
        half = V // 2
        lo, hi = -200.0, 0.0                                   # exp(-200) has integer weight 0
        p = np.array([hi] * half + [lo] * (V - half))
        q = np.array([lo] * half + [hi] * (V - half))
        Ip, Iq = integer_weights(p, 1.0), integer_weights(q, 1.0)
        assert Ip[0] == 1 << 40 and Ip[-1] == 0 and Iq[0] == 0 and Iq[-1] == 1 << 40
        Zp, Zq = sum(Ip), sum(Iq)
        total = sum(max(0, ip * Zq - iq * Zp) >> 48 for ip, iq in zip(Ip, Iq))
        assert total == half * (V - half) << 32
        assert (total < 1 << 64) == fits


def test_eq1_reproduces_paper_tables(golden_dir):
    """Eq. 1 with L_acc + 1 = Tok./Iter, t_t = 1 / AR tok/s and Table 3's t_d gives Table 1's 70B/32K column."""
    rows = [l.split() for l in open(os.path.join(golden_dir, "paper_tables_70b_32k.txt")) if l[0] != "#" and l.strip()]
    ar = next(float(r[2]) for r in rows if r[0] == "AR")
    t_t = 1.0 / ar
    for name, tpi, tps, spd, td_ms in rows:
        if name == "AR":
            continue
        tpi, tps, spd, t_d = float(tpi), float(tps), float(spd), float(td_ms) * 1e-3
        # five of the six rows agree with Eq. 1 to 0.3 %; the table's "Ours 8x L3B" row is 2.8 % off
        # (the paper's own figures for that row do not satisfy Eq. 1 exactly), so it gets 3 %
        tol = 0.03 if name == "Ours8x_L3B" else 0.004
        assert abs(oracle.tokens_per_second(tpi, 5, t_d, t_t) / tps - 1) < tol, name
        assert abs(oracle.sd_speedup(tpi - 1, 5, t_d, t_t) / spd - 1) < tol + 0.003, name
        assert abs(oracle.sd_speedup(tpi - 1, 5, t_d, t_t) - oracle.tokens_per_second(tpi, 5, t_d, t_t) / ar) < 1e-12
    # limiting cases of Eq. 1
    assert oracle.sd_speedup(0, 5, 0.0, 1.0) == 1.0
    assert oracle.sd_speedup(5, 5, 0.0, 1.0) == 6.0
    assert abs(oracle.sd_speedup(4, 5, 1.0, 1.0) - 5 / 6) < 1e-15
