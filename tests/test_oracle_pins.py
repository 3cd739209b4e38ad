"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU needed).

Each test is chosen so that a plausible mistake in the oracle (a dropped term, a wrong sign or index,
a transposed operand, an off-by-one in the window or in the schedule) fails at least one of them.
"""
import math
import os
import subprocess
import sys

import numpy as np
import pytest
from scipy.special import expit, log_expit

import oracle
from oracle import Oracle, StalenessBook
from paper_2211_10280_b200 import synth

LN2 = math.log(2.0)


# ------------------------------------------------------------------ Philox
def test_philox_known_answers(golden_dir):
    n = 0
    for line in open(golden_dir / "philox4x32_10_kat.txt"):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        assert oracle.philox4x32_10(w[:4], w[4:6]) == w[6:]
        n += 1
    assert n == 3


def test_philox_counter_words_are_not_interchangeable():
    # every counter and key word matters, and in its own position
    base = oracle.philox4x32_10([1, 2, 3, 4], [5, 6])
    seen = {tuple(base)}
    for pos in range(4):
        c = [1, 2, 3, 4]
        c[pos] ^= 1
        seen.add(tuple(oracle.philox4x32_10(c, [5, 6])))
    seen.add(tuple(oracle.philox4x32_10([2, 1, 3, 4], [5, 6])))
    seen.add(tuple(oracle.philox4x32_10([1, 2, 3, 4], [6, 5])))
    assert len(seen) == 7


# ------------------------------------------------------------------ alias table
def _alias_mass(thresh, alias):
    """Probability mass of every outcome, in units of 2^-32 / V, as exact Python integers."""
    V = thresh.size
    mass = [0] * V
    for i in range(V):
        t = int(thresh[i])
        if t == 0xFFFFFFFF:
            mass[i] += 1 << 32
        else:
            mass[i] += t
            mass[int(alias[i])] += (1 << 32) - t
    return mass


@pytest.mark.parametrize("V,seed", [(7, 0), (100, 1), (5000, 2)])
def test_alias_reconstructs_count_pow_075(V, seed):
    rng = np.random.default_rng(seed)
    counts = (rng.zipf(1.3, V).astype(np.uint64) % 100000) + 1
    thresh, alias = oracle.build_alias(counts)
    mass = _alias_mass(thresh, alias)
    assert sum(mass) == V << 32
    w = counts.astype(np.float64) ** 0.75
    want = w * V / w.sum() * 2.0 ** 32
    # floor() quantisation loses < 1 unit per small entry; an outcome collects at most V of them
    assert np.max(np.abs(np.array(mass, dtype=np.float64) - want)) <= V + 1e-6 * want.max()
    assert np.all(alias < V)


def test_alias_targets_are_heavy_and_heavy_entries_chain_forward():
    rng = np.random.default_rng(5)
    V = 3000
    counts = (rng.zipf(1.2, V).astype(np.uint64) % 50000) + 1
    thresh, alias = oracle.build_alias(counts)
    w = counts.astype(np.float64) ** 0.75
    mean = w.mean()
    partial = thresh != 0xFFFFFFFF
    assert partial.any() and not partial.all()
    # whatever tops up a bucket has at least the mean weight (the quantisation moves the border by < 1e-9)
    assert np.all(w[alias[partial]] >= mean * (1 - 1e-9))
    # a light entry keeps its own share: thresh / 2^32 = w_i / mean, to the 32-bit floor
    light = partial & (w < mean * (1 - 1e-9))
    np.testing.assert_allclose(thresh[light] / 2.0 ** 32, w[light] / mean, rtol=0, atol=2e-9)
    # a heavy entry whose bucket is topped up is topped up by a later heavy entry
    heavy_partial = partial & (w > mean * (1 + 1e-9))
    assert np.all(alias[heavy_partial] > np.flatnonzero(heavy_partial))
    assert np.array_equal(alias[~partial], np.flatnonzero(~partial))


def test_alias_equal_counts_accept_always():
    thresh, alias = oracle.build_alias(np.full(64, 9, dtype=np.uint64))
    assert np.all(thresh == 0xFFFFFFFF)
    assert np.array_equal(alias, np.arange(64, dtype=np.uint32))


def test_alias_two_outcomes_by_hand():
    # counts 1 and 16 -> weights 1 and 8 -> scaled p = 2/9 and 16/9: slot 0 keeps 2/9, rest goes to 1
    thresh, alias = oracle.build_alias(np.array([1, 16], dtype=np.uint64))
    assert int(thresh[0]) == (2 << 32) // 9 and int(alias[0]) == 1
    assert int(thresh[1]) == 0xFFFFFFFF


def test_draws_follow_unigram_pow_075_chi_square():
    V, k = 50, 8
    counts = (np.arange(V, dtype=np.uint64)[::-1] + 1) ** 2
    o = Oracle(V=V, d=2, window=2, k=k, batch=256, counts=counts, seed=11)
    hist = np.zeros(V)
    rng = np.random.default_rng(0)
    for b in range(40):
        rc, _, _ = o.train_batch(0, rng.integers(0, V, 256), b)
        assert rc == 0
        hist += np.bincount(o.read_negatives().ravel(), minlength=V)
    p = counts.astype(np.float64) ** 0.75
    p /= p.sum()
    n = hist.sum()
    chi2 = float(((hist - n * p) ** 2 / (n * p)).sum())
    # 49 degrees of freedom: mean 49, sd ~9.9; 120 is beyond 7 sigma
    assert n == 40 * synth.n_pairs(256, 2) * k
    assert chi2 < 120.0, chi2


def test_negative_draw_uses_both_halves_of_a_philox_call():
    counts = np.arange(1, 1001, dtype=np.uint64)
    thresh, alias = oracle.build_alias(counts)
    seed, rep, b, p = 0x1234567890ABCDEF, 3, 77, 41
    for j in range(6):
        out = oracle.philox4x32_10([p, j >> 1, b, (1 << 24) | rep], [seed & 0xFFFFFFFF, seed >> 32])
        ra, rb = (out[2], out[3]) if j & 1 else (out[0], out[1])
        slot = (ra * 1000) >> 32
        want = slot if (thresh[slot] == 0xFFFFFFFF or rb < thresh[slot]) else int(alias[slot])
        assert oracle.negative(seed, rep, b, p, j, thresh, alias) == want


# ------------------------------------------------------------------ pairs
def _pairs_brute(tokens, w):
    n = len(tokens)
    return [(q, c) for q in range(n) for c in range(q - w, q + w + 1) if 0 <= c < n and c != q]


@pytest.mark.parametrize("n,w", [(0, 2), (1, 2), (2, 5), (3, 1), (5, 5), (6, 5), (7, 3), (11, 5), (12, 5), (40, 5)])
def test_pair_count_matches_enumeration(n, w):
    V = 50
    o = Oracle(V=V, d=2, window=w, k=2, batch=max(n, 1))
    toks = np.arange(n, dtype=np.int32) % V
    rc, loss, nrows = o.train_batch(0, toks, 0)
    assert rc == 0
    brute = _pairs_brute(toks, w)
    assert o.last_pairs() == len(brute) == synth.n_pairs(n, w)
    if n > w:
        assert len(brute) == 2 * w * n - w * (w + 1)
    if n < 2:
        assert nrows == 0 and loss == 0.0


# ------------------------------------------------------------------ gradient: closed forms
def _dense_reference(o, tokens, w, k, V, d, lr, neg, t_in, t_out):
    """Dense fp64 evaluation of one batch from the per-pair closed form; returns loss, new tables, touched ids."""
    g_in = np.zeros((V, d))
    g_out = np.zeros((V, d))
    touched = set()
    loss = 0.0
    for p, (q, c) in enumerate(_pairs_brute(tokens, w)):
        vc = t_in[tokens[q]].astype(np.float64)
        ctx = int(tokens[c])
        uo = t_out[ctx].astype(np.float64)
        s0 = expit(uo @ vc)
        loss -= log_expit(uo @ vc)
        g_in[tokens[q]] += (s0 - 1.0) * uo          # dL/dv_c, positive term
        g_out[ctx] += (s0 - 1.0) * vc               # dL/du_o
        touched.update([int(tokens[q]), V + ctx])
        for j in range(k):
            r = int(neg[p, j])
            if r == ctx:
                continue
            un = t_out[r].astype(np.float64)
            sj = expit(un @ vc)
            loss -= log_expit(-(un @ vc))
            g_in[tokens[q]] += sj * un              # dL/dv_c, negative terms
            g_out[r] += sj * vc                     # dL/du_n
            touched.add(V + r)
    return loss, g_in, g_out, sorted(touched)


def test_single_batch_matches_per_pair_closed_form():
    V, d, w, k, n, lr = 12, 3, 2, 4, 9, 0.05
    t_in, t_out = synth.random_tables(V, d, seed=5, scale=1.0)
    o = Oracle(V=V, d=d, window=w, k=k, batch=n, lr=lr, seed=3, init_in=t_in, init_out=t_out,
               counts=np.arange(1, V + 1, dtype=np.uint64))
    toks = np.array([3, 3, 7, 0, 11, 3, 5, 5, 1], dtype=np.int32)
    rc, loss, nrows = o.train_batch(0, toks, 4)
    assert rc == 0
    neg = o.read_negatives()
    want_loss, g_in, g_out, touched = _dense_reference(o, toks, w, k, V, d, lr, neg, t_in, t_out)
    ids, delta = o.read_message(0, 4)
    assert ids.tolist() == touched and nrows == len(touched)
    assert loss == pytest.approx(want_loss, rel=1e-12)
    lr32 = float(np.float32(lr))
    dense = np.concatenate([g_in, g_out])
    np.testing.assert_allclose(delta, (-lr32 * dense[ids]).astype(np.float32), rtol=2e-7, atol=1e-12)
    new_in, new_out = o.read_embeddings(0, 0), o.read_embeddings(0, 1)
    np.testing.assert_allclose(new_in, t_in - lr32 * g_in, rtol=3e-7, atol=1e-9)
    np.testing.assert_allclose(new_out, t_out - lr32 * g_out, rtol=3e-7, atol=1e-9)


def test_mean_reduction_divides_the_step_by_the_pair_count():
    # same batch under both readings of L(X): the deltas differ by exactly the factor 1/P (up to fp32 rounding)
    V, d, w, k, n, lr = 30, 5, 2, 3, 12, 0.5
    t_in, t_out = synth.random_tables(V, d, seed=6, scale=0.7)
    toks = np.arange(n, dtype=np.int32) * 2 % V
    out = []
    for red in (0, 1):
        o = Oracle(V=V, d=d, window=w, k=k, batch=n, lr=lr, seed=8, init_in=t_in, init_out=t_out, reduction=red)
        rc, loss, _ = o.train_batch(0, toks, 0)
        assert rc == 0
        out.append((loss, *o.read_message(0, 0), o.read_negatives()))
    P = synth.n_pairs(n, w)
    assert out[0][0] == out[1][0]                       # the reported loss is the sum in both cases
    assert np.array_equal(out[0][1], out[1][1]) and np.array_equal(out[0][3], out[1][3])
    np.testing.assert_allclose(out[1][2], out[0][2] / P, rtol=3e-7, atol=0)
    want_loss, g_in, g_out, _ = _dense_reference(None, toks, w, k, V, d, lr, out[1][3], t_in, t_out)
    dense = np.concatenate([g_in, g_out])
    np.testing.assert_allclose(out[1][2], -(lr / P) * dense[out[1][1]], rtol=3e-7, atol=1e-12)


def test_two_tokens_one_negative_by_hand():
    # tokens [a, b], window 1: pairs (a<-b) and (b<-a).  All output rows zero except the ones set here.
    V, d = 4, 2
    t_in = np.zeros((V, d), np.float32)
    t_out = np.zeros((V, d), np.float32)
    t_in[0] = [1.0, 2.0]
    t_in[1] = [-1.0, 0.5]
    t_out[1] = [0.5, -0.25]      # u_b . v_a = 0  -> sigma = 1/2 exactly
    t_out[0] = [2.0, 4.0]        # u_a . v_b = 0  -> sigma = 1/2 exactly
    o = Oracle(V=V, d=d, window=1, k=1, batch=2, lr=0.5, seed=9, init_in=t_in, init_out=t_out)
    rc, loss, _ = o.train_batch(0, np.array([0, 1], np.int32), 0)
    assert rc == 0
    neg = o.read_negatives()
    g = o.read_g()
    # positives: sigma(0) - 1 = -1/2
    assert g[0, 0] == -0.5 and g[1, 0] == -0.5
    want_in = t_in.astype(np.float64).copy()
    want_out = t_out.astype(np.float64).copy()
    terms = 2
    for p, (c, ctx) in enumerate([(0, 1), (1, 0)]):
        want_in[c] -= 0.5 * (-0.5) * t_out[ctx]
        want_out[ctx] -= 0.5 * (-0.5) * t_in[c]
        r = int(neg[p, 0])
        if r != ctx:
            x = float(t_out[r].astype(np.float64) @ t_in[c].astype(np.float64))
            s = 1.0 / (1.0 + math.exp(-x))
            assert g[p, 1] == pytest.approx(s, rel=1e-7)
            want_in[c] -= 0.5 * s * t_out[r]
            want_out[r] -= 0.5 * s * t_in[c]
            terms += 1 if x == 0.0 else 0
        else:
            assert g[p, 1] == 0.0
    np.testing.assert_allclose(o.read_embeddings(0, 0), want_in, rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(o.read_embeddings(0, 1), want_out, rtol=1e-6, atol=1e-7)
    assert loss >= 2 * LN2


@pytest.mark.parametrize("wl", [synth.scaled(synth.TINY, batches=1),
                                synth.scaled(synth.MID, V=20000, batch=1024, batches=1)])
def test_first_batch_closed_form(wl):
    """With zero output rows every dot product is 0 and every sigmoid is 1/2."""
    toks = synth.token_stream(wl, 0)[0]
    counts = synth.stream_counts([toks], wl.V)
    t_in, _ = synth.init_tables(wl.V, wl.d, 123)
    o = Oracle(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch, lr=wl.lr, seed=wl.seed,
               counts=counts, init_in=t_in)
    rc, loss, nrows = o.train_batch(0, toks, 0)
    assert rc == 0
    neg = o.read_negatives()
    pairs = np.array(_pairs_brute(toks, wl.window))
    assert len(pairs) == wl.pairs_per_batch
    centre, ctx = toks[pairs[:, 0]], toks[pairs[:, 1]]
    live = neg != ctx[:, None].astype(np.uint32)
    assert loss == pytest.approx((len(pairs) + int(live.sum())) * LN2, rel=1e-12)
    # input table bit-unchanged (all deltas are -lr * 0)
    assert np.array_equal(o.read_embeddings(0, 0).view(np.uint32), t_in.view(np.uint32))
    lr32 = float(np.float32(wl.lr))
    want = np.zeros((wl.V, wl.d))
    np.add.at(want, ctx, 0.5 * lr32 * t_in[centre].astype(np.float64))
    for j in range(wl.k):
        m = live[:, j]
        np.add.at(want, neg[m, j], -0.5 * lr32 * t_in[centre[m]].astype(np.float64))
    got = o.read_embeddings(0, 1)
    np.testing.assert_allclose(got, want, rtol=2e-7, atol=1e-12)
    touched_out = set(ctx.tolist()) | set(neg[live].tolist())
    ids, _ = o.read_message(0, 0)
    assert ids.tolist() == sorted(set(centre.tolist())) + [wl.V + r for r in sorted(touched_out)]
    assert nrows == ids.size


def test_gradient_matches_central_finite_differences():
    V, d, w, k, n, lr = 8, 4, 2, 3, 6, 0.25
    rng = np.random.default_rng(42)
    # entries on a 2^-10 grid so that +-h is exact in fp32
    t_in = (rng.integers(-1024, 1024, (V, d)) / 1024.0).astype(np.float32)
    t_out = (rng.integers(-1024, 1024, (V, d)) / 1024.0).astype(np.float32)
    toks = np.array([1, 5, 1, 0, 7, 2], dtype=np.int32)
    o = Oracle(V=V, d=d, window=w, k=k, batch=n, lr=lr, seed=77, init_in=t_in, init_out=t_out)
    h = 2.0 ** -9
    fd = np.zeros((2, V, d))
    for which, tab in ((0, t_in), (1, t_out)):
        for r in range(V):
            for e in range(d):
                row = tab[r:r + 1].copy()
                row[0, e] = tab[r, e] + np.float32(h)
                o.write_embeddings(0, which, r, row)
                lp = o.batch_loss(0, toks, 3)
                row[0, e] = tab[r, e] - np.float32(h)
                o.write_embeddings(0, which, r, row)
                lm = o.batch_loss(0, toks, 3)
                o.write_embeddings(0, which, r, tab[r:r + 1])
                fd[which, r, e] = (lp - lm) / (2 * h)
    rc, loss, _ = o.train_batch(0, toks, 3)
    assert rc == 0
    ids, delta = o.read_message(0, 3)
    grad = np.zeros((2 * V, d))
    grad[ids] = -delta.astype(np.float64) / lr
    fd = fd.reshape(2 * V, d)
    assert np.max(np.abs(fd)) > 0.1
    np.testing.assert_allclose(grad, fd, rtol=0, atol=2e-5)
    # rows outside the message have zero finite difference too
    mask = np.ones(2 * V, bool)
    mask[ids] = False
    assert np.all(fd[mask] == 0.0)


# ------------------------------------------------------------------ message invariants
def test_message_covers_exactly_touched_rows_and_rest_is_bit_unchanged():
    wl = synth.scaled(synth.TINY, V=3000, batches=3)
    stream = synth.token_stream(wl, 0)
    t_in, t_out = synth.random_tables(wl.V, wl.d, 8, scale=0.3)
    o = Oracle(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch, lr=wl.lr, seed=5,
               counts=synth.stream_counts([stream], wl.V), init_in=t_in, init_out=t_out)
    for b in range(3):
        before_in, before_out = o.read_embeddings(0, 0), o.read_embeddings(0, 1)
        rc, _, nrows = o.train_batch(0, stream[b], b)
        assert rc == 0
        neg = o.read_negatives()
        pairs = np.array(_pairs_brute(stream[b], wl.window))
        ctx = stream[b][pairs[:, 1]]
        live = neg != ctx[:, None].astype(np.uint32)
        want = sorted(set(stream[b].tolist())) + [wl.V + r for r in sorted(set(ctx.tolist()) | set(neg[live].tolist()))]
        ids, delta = o.read_message(0, b)
        assert ids.tolist() == want and np.all(np.diff(ids.astype(np.int64)) > 0)
        after = np.concatenate([o.read_embeddings(0, 0), o.read_embeddings(0, 1)])
        before = np.concatenate([before_in, before_out])
        untouched = np.ones(2 * wl.V, bool)
        untouched[ids] = False
        assert np.array_equal(after[untouched].view(np.uint32), before[untouched].view(np.uint32))
        assert np.array_equal(after[ids], before[ids] + delta)   # one fp32 addition per element


def test_masked_negative_contributes_nothing():
    # V = 2 with a huge count on token 1: nearly every draw for a pair whose context is 1 is masked
    V, d = 2, 2
    t_in = np.array([[0.5, -1.0], [0.25, 0.75]], np.float32)
    t_out = np.array([[1.0, 1.0], [-0.5, 2.0]], np.float32)
    o = Oracle(V=V, d=d, window=1, k=6, batch=2, lr=0.1, seed=1, init_in=t_in, init_out=t_out,
               counts=np.array([1, 10 ** 9], np.uint64))
    rc, loss, _ = o.train_batch(0, np.array([0, 1], np.int32), 0)
    neg, g = o.read_negatives(), o.read_g()
    assert np.all(neg[0] == 1)           # pair 0: centre 0, context 1: every draw hits the context
    assert np.all(g[0, 1:] == 0.0)
    x = float(t_out[1].astype(np.float64) @ t_in[0].astype(np.float64))
    # pair 1 (centre 1, context 0) keeps its negatives on row 1
    y = float(t_out[1].astype(np.float64) @ t_in[1].astype(np.float64))
    z = float(t_out[0].astype(np.float64) @ t_in[1].astype(np.float64))
    n1 = int(np.sum(neg[1] == 1))
    want = -log_expit(x) - log_expit(z) - n1 * log_expit(-y)
    assert loss == pytest.approx(want, rel=1e-12)


def test_bad_token_changes_nothing():
    o = Oracle(V=10, d=2, window=1, k=1, batch=4)
    before = o.read_embeddings(0, 0)
    rc, _, _ = o.train_batch(0, np.array([1, 10, 2, 3], np.int32), 0)
    assert rc == -1
    rc, _, _ = o.train_batch(0, np.array([1, -1, 2, 3], np.int32), 0)
    assert rc == -1
    assert np.array_equal(before, o.read_embeddings(0, 0))
    assert np.all(o.sampler()[2] == 1)


def test_seeded_init_is_uniform_in_half_over_d():
    V, d = 4000, 16
    t = oracle.init_input_table(99, V, d)
    assert t.dtype == np.float32 and np.all(np.abs(t) < 0.5 / d)
    assert abs(float(t.mean())) < 3 * (1.0 / d) / math.sqrt(12 * V * d)
    assert float(t.std()) == pytest.approx((1.0 / d) / math.sqrt(12), rel=0.02)
    assert len(np.unique(t)) > 0.99 * V * d
    o = Oracle(V=V, d=d, window=1, k=1, batch=4, W=2, seed=99)
    assert np.array_equal(o.read_embeddings(1, 0), t) and not o.read_embeddings(1, 1).any()


# ------------------------------------------------------------------ DASGD protocol
def test_fig2_staleness_values(golden_dir):
    want = {}
    for line in open(golden_dir / "fig2_staleness.txt"):
        if line.startswith("#") or not line.strip():
            continue
        ev, model, grad, val = line.split()
        want[(ev, grad)] = int(val)
    book = StalenessBook(3)   # models 1, 2, 3 -> indices 0, 1, 2
    red = book.compute(0)
    blue = book.compute(1)
    green = book.compute(2)
    yellow = book.compute(1)
    assert want[("local_apply", "blue")] == 0     # local application has staleness 0 by definition
    assert book.size(1) == want[("size_before_apply", "green")]
    assert book.apply(1, green) == want[("staleness", "green")]
    assert book.size(1) == want[("size_before_apply", "red")]
    assert book.apply(1, red) == want[("staleness", "red")]
    assert {blue, yellow} == {1, 3}


def test_single_replica_is_plain_sgd():
    wl = synth.scaled(synth.TINY, V=500, batches=4)
    stream = synth.token_stream(wl, 0)
    o = Oracle(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch, W=1, max_delay=2)
    for b in range(4):
        assert o.train_batch(0, stream[b], b)[0] == 0
        assert o.apply_messages(0, b) == 0 and o.pending(0) == 0
    assert o.drain() == 0 and o.delivery_log(0).shape[0] == 0


def _run_dasgd(W, max_delay, steps, seed=21, V=400, d=8):
    wl = synth.scaled(synth.TINY, V=V, d=d, batch=64, W=W, batches=steps, stream_seeds=tuple(range(50, 50 + W)),
                      max_delay=max_delay)
    streams = synth.all_streams(wl)
    t_in, t_out = synth.random_tables(V, d, 2, scale=0.2)
    o = Oracle(V=V, d=d, window=wl.window, k=wl.k, batch=wl.batch, W=W, lr=wl.lr, max_delay=max_delay,
               seed=seed, counts=synth.stream_counts(streams, V), init_in=t_in, init_out=t_out)
    msgs = {}
    for t in range(steps):
        for i in range(W):
            assert o.train_batch(i, streams[i][t], t)[0] == 0
            msgs[(i, t)] = o.read_message(i, t)
        for j in range(W):
            o.apply_messages(j, t)
    return o, msgs, (t_in, t_out)


def test_every_message_is_delivered_once_in_order_and_within_the_delay_bound():
    W, D, T = 4, 2, 12
    o, msgs, _ = _run_dasgd(W, D, T)
    delays = set()
    for j in range(W):
        log = o.delivery_log(j)
        prev = None
        for origin, sender, due, at, _ in log.tolist():
            assert sender != j and due == at and 0 <= due - origin <= D
            assert due == origin + o.delay(origin, sender, j)
            delays.add(due - origin)
            if prev is not None and prev[0] == at:
                assert (prev[1], prev[2]) < (origin, sender)    # (origin step, sender) order in a step
            prev = (at, origin, sender)
    assert delays == {0, 1, 2}
    pending = sum(o.pending(j) for j in range(W))
    assert o.drain() == pending
    for j in range(W):
        log = o.delivery_log(j)
        got = sorted((int(s), int(t)) for t, s, *_ in log.tolist())
        assert got == sorted((i, t) for i in range(W) if i != j for t in range(T))


def test_staleness_log_matches_set_arithmetic():
    W, D, T = 3, 2, 8
    o, _, _ = _run_dasgd(W, D, T)
    o.drain()
    G = [set() for _ in range(W)]
    snap = {}
    inbox = [[] for _ in range(W)]
    want = [[] for _ in range(W)]
    for t in range(T):
        for i in range(W):
            snap[(i, t)] = set(G[i])
            G[i].add((i, t))
            for j in range(W):
                if j != i:
                    inbox[j].append((t + o.delay(t, i, j), t, i))
        for j in range(W):
            due = sorted([x for x in inbox[j] if x[0] <= t], key=lambda x: (x[1], x[2]))
            inbox[j] = [x for x in inbox[j] if x[0] > t]
            for _, ot, s in due:
                want[j].append(len(snap[(s, ot)] ^ G[j]))
                G[j].add((s, ot))
    for j in range(W):
        for _, ot, s in sorted(inbox[j]):
            want[j].append(len(snap[(s, ot)] ^ G[j]))
            G[j].add((s, ot))
        assert o.delivery_log(j)[:, 4].tolist() == want[j]
    assert max(max(w) for w in want) > 0


def test_replicas_agree_after_drain_and_equal_init_plus_all_messages():
    W, D, T = 4, 2, 6
    o, msgs, (t_in, t_out) = _run_dasgd(W, D, T)
    o.drain()
    V = o.V
    total = np.concatenate([t_in, t_out]).astype(np.float64)
    for (i, t), (ids, delta) in msgs.items():
        total[ids] += delta
    ref = np.concatenate([o.read_embeddings(0, 0), o.read_embeddings(0, 1)])
    np.testing.assert_allclose(ref, total, rtol=0, atol=2e-6)
    for j in range(1, W):
        other = np.concatenate([o.read_embeddings(j, 0), o.read_embeddings(j, 1)])
        np.testing.assert_allclose(other, ref, rtol=0, atol=2e-6)
    assert not np.array_equal(ref[:V], t_in)


def test_zero_delay_keeps_replicas_in_lockstep():
    # with every delay 0 all replicas hold theta + sum_i delta_i(theta) after each step:
    # N models with batch b behave like one model with batch N*b
    W, T = 3, 3
    o, msgs, (t_in, t_out) = _run_dasgd(W, 0, T)
    for j in range(W):
        assert o.pending(j) == 0 and np.all(o.delivery_log(j)[:, 2] == o.delivery_log(j)[:, 0])
    a = o.read_embeddings(0, 1)
    for j in range(1, W):
        np.testing.assert_allclose(o.read_embeddings(j, 1), a, rtol=0, atol=1e-6)


def test_loss_starts_at_ln2_per_term_and_decreases():
    wl = synth.TINY
    stream = synth.token_stream(wl, 0)
    o = Oracle(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch, lr=wl.lr, seed=wl.seed,
               counts=synth.stream_counts([stream], wl.V))
    losses = [o.train_batch(0, stream[b], b)[1] for b in range(60)]
    P = wl.pairs_per_batch
    assert losses[0] <= P * (1 + wl.k) * LN2 and losses[0] > P * (1 + wl.k) * LN2 * 0.99
    assert np.mean(losses[-10:]) < 0.95 * losses[0]


def test_result_does_not_depend_on_thread_count(tmp_path):
    code = (
        "import sys, numpy as np; sys.path.insert(0, %r)\n"
        "from oracle import Oracle\n"
        "from paper_2211_10280_b200 import synth\n"
        "wl = synth.scaled(synth.TINY, V=2000, batches=2)\n"
        "s = synth.token_stream(wl, 0)\n"
        "o = Oracle(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch, seed=3)\n"
        "l = [o.train_batch(0, s[b], b)[1] for b in range(2)]\n"
        "np.save(sys.argv[1], np.concatenate([o.read_embeddings(0,0).ravel(), o.read_embeddings(0,1).ravel(), l]))\n"
    ) % str(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    outs = []
    for nt in ("1", "4"):
        f = tmp_path / f"t{nt}.npy"
        env = dict(os.environ, OMP_NUM_THREADS=nt)
        subprocess.check_call([sys.executable, "-c", code, str(f)], env=env)
        outs.append(np.load(f))
    assert np.array_equal(outs[0].view(np.uint64), outs[1].view(np.uint64))


# ------------------------------------------------------------------ drift metric
def test_cosine_difference_special_cases_and_library_formula():
    rng = np.random.default_rng(3)
    a = rng.standard_normal((50, 7)).astype(np.float32)
    b = rng.standard_normal((50, 7)).astype(np.float32)
    got = oracle.cosine_difference(a, b)
    a64, b64 = a.astype(np.float64), b.astype(np.float64)
    want = 1.0 - np.einsum("ij,ij->i", a64, b64) / (np.linalg.norm(a64, axis=1) * np.linalg.norm(b64, axis=1))
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-7)
    assert np.all(oracle.cosine_difference(a, 3.5 * a) < 1e-7)                    # same direction, any length
    np.testing.assert_allclose(oracle.cosine_difference(a, -a), 2.0, atol=1e-7)   # opposite
    e = np.eye(4, dtype=np.float32)
    np.testing.assert_allclose(oracle.cosine_difference(e, np.roll(e, 1, axis=0)), 1.0, atol=0)   # orthogonal
    z = np.zeros((2, 4), np.float32)
    assert oracle.cosine_difference(z, z).tolist() == [0.0, 0.0]
    assert oracle.cosine_difference(z, e[:2]).tolist() == [1.0, 1.0]


def test_top_drifted_rows_against_a_library_sort_brute_force_and_special_values():
    rng = np.random.default_rng(11)
    # distinct finite values: the library's argsort of the negated values is the definition
    x = rng.permutation(5000).astype(np.float32) / 7.0 - 200.0
    ids, vals = oracle.top_drifted(x, 37)
    want = np.argsort(-x.astype(np.float64), kind="stable")[:37]
    assert ids.tolist() == want.tolist() and np.array_equal(vals, x[want])
    # heavy ties: equal values come out in ascending row order (lexsort: last key is the primary one)
    y = rng.integers(0, 6, 2000).astype(np.float32) * 0.25
    for k in (1, 5, 400, 1999, 2000, 5000):
        ids, vals = oracle.top_drifted(y, k)
        want = np.lexsort((np.arange(y.size), -y))[:k]
        assert ids.tolist() == want.tolist() and np.array_equal(vals, y[want])
    # brute force on tiny inputs: repeatedly take the maximum, the first one among equals
    for n in range(0, 7):
        z = rng.integers(-2, 3, n).astype(np.float32)
        left = list(range(n))
        want = []
        while left:
            best = max(left, key=lambda i: (z[i], -i))
            want.append(best)
            left.remove(best)
        for k in range(0, n + 2):
            assert oracle.top_drifted(z, k)[0].tolist() == want[:k]
    # the total order of the bit patterns: +NaN above +inf, -0 below +0, -NaN lowest
    s = np.array([0.0, -0.0, np.inf, -np.inf, 1.0, np.nan, -1.0, 0.0], np.float32)
    s[5] = np.frombuffer(np.uint32(0x7FC00000).tobytes(), np.float32)[0]
    neg_nan = np.frombuffer(np.uint32(0xFFC00000).tobytes(), np.float32)[0]
    s = np.append(s, neg_nan).astype(np.float32)
    assert oracle.top_drifted(s, 9)[0].tolist() == [5, 2, 4, 0, 7, 1, 6, 3, 8]


# ------------------------------------------------------------------ routed mini-batches (hash partition by centre word)
def test_route_is_a_partition_of_the_vocabulary_and_roughly_even():
    for W in (1, 2, 3, 8):
        r = np.array([oracle.route(77, W, x) for x in range(6000)])
        assert r.min() == 0 and r.max() == W - 1
        share = np.bincount(r, minlength=W) / r.size
        assert np.all(np.abs(share - 1.0 / W) < 0.03)
    assert [oracle.route(77, 5, x) for x in range(50)] == [oracle.route(77, 5, x) for x in range(50)]
    assert [oracle.route(77, 5, x) for x in range(50)] != [oracle.route(78, 5, x) for x in range(50)]


@pytest.mark.parametrize("reduction", [0, 1])
def test_routed_parts_of_a_minibatch_add_up_to_the_gradient_of_the_whole_batch(reduction):
    # Section 4.3: pairs are spread over the Model instances by the hash of x.  The parts are disjoint
    # sets of pairs of one batch, so they must add up to what a single model computes from that batch.
    V, d, W, w, k = 200, 6, 3, 3, 4
    wl = synth.scaled(synth.TINY, V=V, d=d, window=w, k=k, batch=64, batches=2)
    stream = synth.token_stream(wl, 0)
    counts = synth.stream_counts([stream], V)
    t_in, t_out = synth.random_tables(V, d, 8, scale=0.4)
    kw = dict(V=V, d=d, window=w, k=k, batch=64, lr=0.05, seed=21, counts=counts, init_in=t_in, init_out=t_out,
              reduction=reduction)
    solo, many = Oracle(W=1, **kw), Oracle(W=W, max_delay=0, **kw)
    for b in range(2):
        toks = stream[b]
        rc, loss_solo, _ = solo.train_batch(0, toks, b)
        assert rc == 0
        neg_solo, g_solo = solo.read_negatives(), solo.read_g()
        ids_solo, delta_solo = solo.read_message(0, b)
        before = [many.read_embeddings(r, 0).copy() for r in range(W)]
        losses, owners, g_sum = [], np.zeros(neg_solo.shape[0], int), np.zeros_like(g_solo)
        summed = np.zeros((2 * V, d))
        seen_in = set()
        for r in range(W):
            rc, loss_r, _ = many.train_batch_routed(r, toks, b)
            assert rc == 0
            losses.append(loss_r)
            neg_r, g_r = many.read_negatives(), many.read_g()
            own = neg_r[:, 0] != 0xFFFFFFFF
            assert np.array_equal(neg_r[own], neg_solo[own])                     # the whole batch's draws
            assert np.all(g_r[~own] == 0.0)
            if b == 0:
                assert np.array_equal(g_r[own], g_solo[own])
            owners += own
            g_sum += g_r
            ids_r, delta_r = many.read_message(r, b)
            ins = ids_r[ids_r < V]
            assert all(oracle.route(21, W, int(x)) == r for x in ins)           # only its own centre words
            assert not (set(ins.tolist()) & seen_in)
            seen_in |= set(ins.tolist())
            summed[ids_r] += delta_r
            # rows outside its message are untouched by its own step
            after = many.read_embeddings(r, 0)
            mask = np.ones(V, bool)
            mask[ins] = False
            assert np.array_equal(after[mask], before[r][mask])
        assert np.all(owners == 1)                                               # every pair trained exactly once
        # batch 0 starts from identical tables; later the replicas differ from the single model by fp32 rounding order
        assert sum(losses) == pytest.approx(loss_solo, rel=1e-12 if b == 0 else 1e-6)
        if b == 0:
            np.testing.assert_array_equal(g_sum, g_solo)
            touched = np.flatnonzero(np.abs(summed).sum(axis=1) > 0)
            assert set(touched.tolist()) <= set(ids_solo.tolist())
            np.testing.assert_allclose(summed[ids_solo], delta_solo, rtol=0, atol=3e-7 * np.abs(delta_solo).max())
        for r in range(W):
            assert many.apply_messages(r, b) == W - 1
        if b == 0:
            for r in range(W):
                for which in (0, 1):
                    np.testing.assert_allclose(many.read_embeddings(r, which), solo.read_embeddings(0, which),
                                               rtol=0, atol=2e-7)
    # the running unigram counts saw every token once
    assert np.array_equal(many.sampler()[2], solo.sampler()[2])


# ------------------------------------------------------------------ maxGradBuffer > 1
def test_buffered_gradients_are_summed_over_the_union_of_their_rows_and_sent_every_mth_batch():
    # Algorithm 1: every gradient joins the buffer; the buffer is sent when it holds maxGradBuffer gradients.
    V, d, m, T = 300, 6, 3, 7
    wl = synth.scaled(synth.TINY, V=V, d=d, batch=48, batches=T)
    stream = synth.token_stream(wl, 0)
    t_in, t_out = synth.random_tables(V, d, 4, scale=0.3)
    kw = dict(V=V, d=d, window=wl.window, k=wl.k, batch=wl.batch, lr=0.05, seed=9, init_in=t_in, init_out=t_out)
    solo = Oracle(W=1, **kw)                               # the same trajectory, every batch message visible
    pair = Oracle(W=2, max_delay=0, max_grad_buffer=m, **kw)   # replica 1 never trains, so replica 0 receives nothing
    per_batch = []
    for t in range(T):
        assert solo.train_batch(0, stream[t], t)[0] == 0
        per_batch.append(solo.read_message(0, t))
        assert pair.train_batch(0, stream[t], t)[0] == 0
        applied = pair.apply_messages(1, t)
        assert applied == (1 if t % m == m - 1 else 0)     # m times fewer messages
        if t % m == m - 1:
            ids, delta = pair.read_message(0, t)
            want = {}
            for bi, bd in per_batch[-m:]:
                for r, i in enumerate(bi.tolist()):
                    want[i] = bd[r].copy() if i not in want else (want[i] + bd[r]).astype(np.float32)
            assert ids.tolist() == sorted(want)
            assert np.array_equal(delta, np.stack([want[i] for i in ids.tolist()]))
        else:
            assert pair.read_message(0, t) is None
    assert np.array_equal(pair.read_embeddings(0, 1), solo.read_embeddings(0, 1))
    # the receiver holds init + the two merged messages; the 7th batch is still buffered at the sender
    log = pair.delivery_log(1)
    assert log[:, 0].tolist() == [2, 5] and pair.drain() == 0
