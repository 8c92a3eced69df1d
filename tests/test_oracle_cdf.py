"""Pins for the oracle's CDF-threshold mask mode (Section 8.1): the fixed-arithmetic 2^x against the
library's, the kept set against an fp64 sorted-cumulative-mass definition, closed-form cases."""
import numpy as np


def _bits(words, NB):
    return {j for j in range(NB) if (int(words[j >> 5]) >> (j & 31)) & 1}


def test_exp2c_matches_library_exp2(oracle_mod):
    x = np.concatenate([np.linspace(-125, 0, 200001), -np.logspace(-6, 2, 2000), [0.0, -0.5, -1.5, -2.5, -124.5]]).astype(np.float32)
    y = oracle_mod.exp2c(x)
    ref = np.exp2(x.astype(np.float64))
    assert np.abs(y / ref - 1.0).max() < 4e-7
    assert oracle_mod.exp2c(np.array([0.0], np.float32))[0] == np.float32(1.0000001192092896)  # the constant term
    assert np.all(oracle_mod.exp2c(np.array([-300.0, -1e30], np.float32)) == oracle_mod.exp2c(np.array([-125.0], np.float32))[0])
    assert np.all(np.diff(oracle_mod.exp2c(np.linspace(-30, 0, 100001).astype(np.float32)).astype(np.float64)) >= 0)  # monotone


def _f64_reference_sets(srow, cand, tau, scale):
    """Smallest top set by score (whole tie groups) whose fp64 softmax mass reaches tau; also the mass of that set
    and of the set without its lowest group."""
    s = srow[cand].astype(np.float64) * scale
    p = np.exp(s - s.max())
    p /= p.sum()
    order = np.argsort(-s, kind="stable")
    vals = s[order]
    cum = 0.0
    t = 0
    prev = 0.0
    while t < len(order):
        v = vals[t]
        prev = cum
        while t < len(order) and vals[t] == v:
            cum += p[order[t]]
            t += 1
        if cum >= tau:
            break
    return {int(cand[j]) for j in order[:t]}, cum, prev


def test_kept_set_is_the_smallest_top_set_reaching_tau(oracle_mod):
    rng = np.random.default_rng(3)
    for (H, NB, n_text_blocks, tau, spread) in [(2, 40, 0, 0.9, 3.0), (1, 97, 2, 0.85, 6.0), (2, 33, 1, 0.95, 1.0), (1, 64, 0, 0.5, 10.0)]:
        sc = (rng.standard_normal((H, NB, NB)) * spread).astype(np.float32)
        is_text = np.zeros(NB, np.uint8)
        if n_text_blocks:
            is_text[-n_text_blocks:] = 1
        scale = 0.37
        mask, cnt = oracle_mod.cdf_mask(sc, is_text, tau, scale)
        cand = np.flatnonzero(is_text == 0)
        for h in range(H):
            for i in range(NB):
                got = _bits(mask[h, i], NB)
                assert {int(j) for j in np.flatnonzero(is_text)} <= got          # text blocks always kept
                got_c = got - {int(j) for j in np.flatnonzero(is_text)}
                assert cnt[h, i] == len(got)
                want, mass, mass_without_last = _f64_reference_sets(sc[h, i], cand, tau, scale)
                if got_c != want:
                    # only a cumulative mass within fp32 rounding of tau may tip the decision
                    assert abs(mass - tau) < 1e-5 or abs(mass_without_last - tau) < 1e-5, (h, i, mass, mass_without_last)
                # a top set by score: every kept score >= every dropped score
                kept_scores = sc[h, i][sorted(got_c)]
                dropped = sorted(set(cand.tolist()) - got_c)
                if dropped:
                    assert kept_scores.min() > sc[h, i][dropped].max()


def test_closed_form_cases(oracle_mod):
    NB = 48
    is_text = np.zeros(NB, np.uint8)
    # (a) all scores equal: one tie group, everything is kept whatever tau
    sc = np.full((1, NB, NB), 1.25, np.float32)
    mask, cnt = oracle_mod.cdf_mask(sc, is_text, 0.3, 1.0)
    assert np.all(cnt == NB)
    # (b) one block carries more than tau of the mass: exactly that block
    sc = np.zeros((1, NB, NB), np.float32)
    for i in range(NB):
        sc[0, i, (7 * i) % NB] = 12.0            # e^12 / (e^12 + 47) = 0.9997
    mask, cnt = oracle_mod.cdf_mask(sc, is_text, 0.95, 1.0)
    assert np.all(cnt == 1)
    for i in range(NB):
        assert _bits(mask[0, i], NB) == {(7 * i) % NB}
    # (c) two levels: n1 blocks at score a, the rest at 0 -> mass of the top group = n1 e^a / (n1 e^a + NB - n1)
    n1, a = 6, 1.0
    sc = np.zeros((1, NB, NB), np.float32)
    sc[0, :, :n1] = a
    top = n1 * np.exp(a) / (n1 * np.exp(a) + NB - n1)      # 0.2797
    mask, cnt = oracle_mod.cdf_mask(sc, is_text, float(top) - 0.01, 1.0)
    assert np.all(cnt == n1)
    mask, cnt = oracle_mod.cdf_mask(sc, is_text, float(top) + 0.01, 1.0)
    assert np.all(cnt == NB)
    # (d) tau = 1 keeps everything that has any mass in fp32; -0.0 and +0.0 tie
    sc = np.zeros((1, NB, NB), np.float32)
    sc[0, :, ::2] = -0.0
    mask, cnt = oracle_mod.cdf_mask(sc, is_text, 1.0, 1.0)
    assert np.all(cnt == NB)


def test_scale_and_text_blocks(oracle_mod):
    rng = np.random.default_rng(5)
    NB = 30
    sc = rng.standard_normal((1, NB, NB)).astype(np.float32)
    is_text = np.zeros(NB, np.uint8)
    is_text[-3:] = 1
    sc[0, :, -3:] = 50.0                          # huge text scores must not take part in the softmax
    m_small, c_small = oracle_mod.cdf_mask(sc, is_text, 0.9, 0.1)   # flat distribution: many blocks
    m_big, c_big = oracle_mod.cdf_mask(sc, is_text, 0.9, 10.0)      # peaked distribution: few blocks
    assert c_small.mean() > c_big.mean() + 5
    assert np.all(c_big >= 4)                     # at least one candidate + the three text blocks


def test_kept_set_does_not_depend_on_block_order(oracle_mod):
    """The mass is an integer sum, so renumbering the key blocks renumbers the kept set and changes nothing else
    (a floating-point sum taken in index order would not guarantee that)."""
    rng = np.random.default_rng(11)
    NB = 75
    sc = (rng.standard_normal((2, NB, NB)) * 2.0).astype(np.float32)
    is_text = np.zeros(NB, np.uint8)
    for tau in (0.5, 0.9, 0.99):
        mask, cnt = oracle_mod.cdf_mask(sc, is_text, tau, 0.5)
        perm = rng.permutation(NB)
        mask_p, cnt_p = oracle_mod.cdf_mask(np.ascontiguousarray(sc[:, :, perm]), is_text, tau, 0.5)
        assert np.array_equal(cnt, cnt_p)
        for h in range(2):
            for i in range(NB):
                assert {int(perm[j]) for j in _bits(mask_p[h, i], NB)} == _bits(mask[h, i], NB)
