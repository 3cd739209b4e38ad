"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs.

Bars: bit-exact for sampled negatives, sampler tables, counts, message row ids, delivery order and
staleness; max relative error (see parity_utils.rel_err) <= 1e-5 for fp32 embeddings and delta rows
after one batch and <= 1e-3 after 200 batches.
"""
import math

import numpy as np
import pytest

from parity_utils import compare_message, compare_tables, make_pair, rel_err
from paper_2211_10280_b200 import synth

pytestmark = pytest.mark.gpu

TOL_ONE = 1e-5
TOL_200 = 1e-3


@pytest.fixture(scope="module")
def torch():
    import torch as t

    assert t.cuda.is_available(), "these tests need a CUDA device"
    return t


def dev(torch, a):
    """The batch in device memory, complete when this returns (so that the suite can also run with the knob that lets
    the library start on a batch's tokens ahead of the stream: TENSAIR_TUNE=early_prepare=2)."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()
    torch.cuda.current_stream().synchronize()
    return t


# ------------------------------------------------------------------ init, sampler
def test_seeded_init_is_bit_identical(torch):
    import oracle as orc

    wl = synth.scaled(synth.TINY, V=3001, d=68, W=2)
    o, g = make_pair(wl)
    want = orc.init_input_table(wl.seed, wl.V, wl.d)
    for r in range(2):
        assert np.array_equal(g.tensair_read_embeddings(r, 0).view(np.uint32), want.view(np.uint32))
        assert not g.tensair_read_embeddings(r, 1).any()
    assert np.array_equal(o.read_embeddings(1, 0), want)


@pytest.mark.parametrize("wl", [synth.TINY, synth.scaled(synth.MID, batches=2),
                                synth.scaled(synth.LARGE_DASGD, V=60_000, d=12, batch=2048, W=1, max_delay=0)],
                         ids=lambda w: w.name)
def test_negatives_sampler_and_counts_are_bit_exact(torch, wl):
    stream = synth.token_stream(wl, 0, 2)
    counts = synth.stream_counts([stream], wl.V)
    o, g = make_pair(wl, counts=counts)
    to, ao, _ = o.sampler()
    tg, ag, _ = g.tensair_read_sampler()
    assert np.array_equal(to, tg) and np.array_equal(ao, ag)
    for b in range(2):
        assert o.train_batch(0, stream[b], b + 5)[0] == 0
        g.tensair_train_batch(0, dev(torch, stream[b]), b + 5)
        no, ng = o.read_negatives(), g.tensair_read_negatives()
        assert no.shape == ng.shape == (wl.pairs_per_batch, wl.k)
        assert np.array_equal(no, ng)
    assert np.array_equal(o.sampler()[2], g.tensair_read_sampler()[2])


# ------------------------------------------------------------------ one batch
ONE_BATCH = [
    ("tiny", synth.TINY, False),
    ("tiny_mean", synth.scaled(synth.TINY, reduction=1), True),
    ("tiny_random_tables", synth.TINY, True),
    ("mid", synth.MID, True),
    ("d300_k15", synth.scaled(synth.LARGE_DASGD, V=50_000, batch=1024, W=1, max_delay=0), True),
    ("d512_k5", synth.scaled(synth.sweep_point(512, 2048, 5), V=30_000), True),
    ("d8_w1_k1", synth.scaled(synth.TINY, V=500, d=8, window=1, k=1, batch=100), True),
    ("d1024_w8_k3", synth.scaled(synth.TINY, V=2000, d=1024, window=8, k=3, batch=300), True),
    ("w16_k2", synth.scaled(synth.TINY, V=3000, d=64, window=16, k=2, batch=600), True),
    ("V2_every_other_negative_dropped", synth.scaled(synth.TINY, V=2, d=8, window=2, k=3, batch=50), True),
    ("k40_d100", synth.scaled(synth.TINY, V=4000, d=100, window=2, k=40, batch=200, reduction=1), True),
    # every width class of the forward kernel: slices of 2 floats in 3 and 7 rounds, slices of 4 in 2 and 3 rounds,
    # with whole 8-row chunks (k = 7, 15), whole 6-row chunks (k = 5) and ragged ones (k = 9)
    ("d192_k7", synth.scaled(synth.TINY, V=3000, d=192, window=3, k=7, batch=300, reduction=1), True),
    ("d448_k5", synth.scaled(synth.TINY, V=3000, d=448, window=2, k=5, batch=300, reduction=1), True),
    ("d256_k15", synth.scaled(synth.TINY, V=3000, d=256, window=2, k=15, batch=300, reduction=1), True),
    ("d384_k9", synth.scaled(synth.TINY, V=3000, d=384, window=2, k=9, batch=300, reduction=1), True),
    ("d36_stride40", synth.scaled(synth.TINY, V=3000, d=36, window=2, k=15, batch=300, reduction=1), True),
]


@pytest.mark.parametrize("name,wl,random_tables", ONE_BATCH, ids=[c[0] for c in ONE_BATCH])
def test_one_batch_matches_the_oracle(torch, name, wl, random_tables):
    stream = synth.token_stream(wl, 0, 1)
    counts = synth.stream_counts([stream], wl.V)
    if random_tables:
        t_in, t_out = synth.random_tables(wl.V, wl.d, 17, scale=2.0 / math.sqrt(wl.d))
    else:
        t_in, t_out = synth.init_tables(wl.V, wl.d, 17)
    o, g = make_pair(wl, counts=counts, init_in=t_in, init_out=t_out)
    rc, loss_o, nrows_o = o.train_batch(0, stream[0], 0)
    assert rc == 0
    loss_g, info = g.tensair_train_batch(0, dev(torch, stream[0]), 0, want_loss=True, want_info=True)
    assert info.n_pairs == wl.pairs_per_batch == o.last_pairs()
    assert info.n_rows == nrows_o
    assert info.n_in_rows == len(set(stream[0].tolist()))
    assert np.array_equal(o.read_negatives(), g.tensair_read_negatives())
    go, gg = o.read_g(), g.tensair_read_scalars()
    assert np.max(np.abs(go - gg)) <= 1e-13
    assert np.array_equal(go == 0.0, gg == 0.0)
    assert loss_g == pytest.approx(loss_o, rel=1e-12)
    compare_message(o, g, 0, 0, TOL_ONE)
    compare_tables(o, g, 0, TOL_ONE)
    # rows outside the message are bit-unchanged
    ids, _ = g.tensair_read_message(0, 0)
    untouched = np.ones(2 * wl.V, bool)
    untouched[ids] = False
    after = np.concatenate([g.tensair_read_embeddings(0, 0), g.tensair_read_embeddings(0, 1)])
    before = np.concatenate([t_in, t_out])
    assert np.array_equal(after[untouched].view(np.uint32), before[untouched].view(np.uint32))
    assert g.tensair_apply_messages(0, 0) == 0


def test_hot_rows_take_the_chunked_path(torch):
    # 40 tokens and a large batch: every row collects far more than one chunk of contributions
    wl = synth.scaled(synth.TINY, V=40, d=36, window=3, k=7, batch=3000, zipf_s=0.3)
    stream = synth.token_stream(wl, 0, 2)
    t_in, t_out = synth.random_tables(wl.V, wl.d, 3, scale=0.05)
    o, g = make_pair(wl, counts=synth.stream_counts([stream], wl.V), init_in=t_in, init_out=t_out)
    for b in range(2):
        assert o.train_batch(0, stream[b], b)[0] == 0
        g.tensair_train_batch(0, dev(torch, stream[b]), b)
        compare_message(o, g, 0, b, TOL_ONE)
    compare_tables(o, g, 0, 3 * TOL_ONE)


def test_batch_of_one_repeated_token(torch):
    # every pair is (x, x): all input and output contributions fall on two rows, and every draw of x
    # as a negative is dropped because it equals the positive context
    wl = synth.scaled(synth.TINY, V=50, d=24, window=4, k=6, batch=400, reduction=1)
    toks = np.full(wl.batch, 7, np.int32)
    t_in, t_out = synth.random_tables(wl.V, wl.d, 5, scale=0.3)
    counts = np.ones(wl.V, np.uint64)
    counts[7] = 1000
    o, g = make_pair(wl, counts=counts, init_in=t_in, init_out=t_out)
    rc, loss_o, nrows_o = o.train_batch(0, toks, 0)
    assert rc == 0
    loss_g, info = g.tensair_train_batch(0, dev(torch, toks), 0, want_loss=True, want_info=True)
    assert info.n_in_rows == 1 and info.n_rows == nrows_o
    neg = g.tensair_read_negatives()
    assert np.array_equal(o.read_negatives(), neg)
    go, gg = o.read_g(), g.tensair_read_scalars()
    assert np.array_equal(go == 0.0, gg == 0.0) and np.max(np.abs(go - gg)) <= 1e-13
    assert loss_g == pytest.approx(loss_o, rel=1e-12)
    compare_message(o, g, 0, 0, TOL_ONE)
    compare_tables(o, g, 0, TOL_ONE)


def test_eight_replicas_with_delays_up_to_three_steps(torch):
    wl = synth.scaled(synth.LARGE_DASGD, V=3000, d=20, batch=128, k=4, W=8, max_delay=3,
                      stream_seeds=tuple(range(40, 48)))
    o, g = _run_exchange(torch, wl, 9)
    assert o.drain() == g.tensair_drain()
    for j in range(wl.W):
        assert np.array_equal(o.delivery_log(j), g.tensair_read_delivery_log(j))
        compare_tables(o, g, j, TOL_200)


@pytest.mark.parametrize("n", [0, 1, 2, 3, 5, 6, 10, 11, 12, 509, 512])
def test_ragged_and_degenerate_batches(torch, n):
    wl = synth.scaled(synth.TINY, V=700, d=20, window=5, k=4)
    toks = synth.token_stream(wl, 0, 1)[0][:n]
    t_in, t_out = synth.random_tables(wl.V, wl.d, 9, scale=0.4)
    o, g = make_pair(wl, init_in=t_in, init_out=t_out)
    rc, loss_o, nrows_o = o.train_batch(0, toks, 3)
    assert rc == 0
    loss_g, info = g.tensair_train_batch(0, dev(torch, toks) if n else torch.empty(0, dtype=torch.int32, device="cuda"),
                                         3, want_loss=True, want_info=True)
    assert info.n_rows == nrows_o and info.n_pairs == synth.n_pairs(n, 5)
    assert loss_g == pytest.approx(loss_o, rel=2e-6, abs=1e-12)
    if n >= 2:
        assert np.array_equal(o.read_negatives(), g.tensair_read_negatives())
        compare_message(o, g, 0, 3, TOL_ONE)
    compare_tables(o, g, 0, TOL_ONE)
    assert np.array_equal(o.sampler()[2], g.tensair_read_sampler()[2])


def test_bad_token_is_reported_and_changes_nothing(torch):
    from paper_2211_10280_b200 import binding as B

    wl = synth.scaled(synth.TINY, V=300, d=16)
    t_in, t_out = synth.random_tables(wl.V, wl.d, 1)
    o, g = make_pair(wl, init_in=t_in, init_out=t_out)
    toks = synth.token_stream(wl, 0, 1)[0].copy()
    bad = toks.copy()
    bad[77] = wl.V
    with pytest.raises(B.TensairError) as ei:
        g.tensair_train_batch(0, dev(torch, bad), 0, want_loss=True)
    assert ei.value.code == B.EBADTOKEN
    assert np.array_equal(g.tensair_read_embeddings(0, 0), t_in) and np.array_equal(g.tensair_read_embeddings(0, 1), t_out)
    assert np.all(g.tensair_read_sampler()[2] == 1)
    bad[77] = -1
    g.tensair_train_batch(0, dev(torch, bad), 1)          # asynchronous: reported by the next sync
    assert g.tensair_sync() == B.EBADTOKEN and g.tensair_sync() == B.OK
    # the context keeps working
    assert o.train_batch(0, toks, 2)[0] == 0
    g.tensair_train_batch(0, dev(torch, toks), 2)
    compare_tables(o, g, 0, TOL_ONE)


def test_host_and_device_entry_points_agree_bit_for_bit(torch):
    wl = synth.scaled(synth.TINY, V=2000, d=32)
    stream = synth.token_stream(wl, 0, 3)
    t_in, t_out = synth.random_tables(wl.V, wl.d, 4, scale=0.3)
    counts = synth.stream_counts([stream], wl.V)
    _, g1 = make_pair(wl, counts=counts, init_in=t_in, init_out=t_out)
    _, g2 = make_pair(wl, counts=counts, init_in=t_in, init_out=t_out)
    pinned = torch.from_numpy(stream).pin_memory()
    for b in range(3):
        l1, _ = g1.tensair_train_batch(0, dev(torch, stream[b]), b, want_loss=True)
        l2, _ = g2.tensair_train_batch_host(0, pinned[b], b, want_loss=True)
        assert l1 == l2
    for which in (0, 1):
        assert np.array_equal(g1.tensair_read_embeddings(0, which).view(np.uint32),
                              g2.tensair_read_embeddings(0, which).view(np.uint32))


def test_loss_read_back_without_waiting_equals_the_blocking_read(torch):
    wl = synth.scaled(synth.MID, V=20_000, batch=1024, W=2, stream_seeds=(1, 2), batches=3)
    streams = synth.all_streams(wl, 3)
    _, g = make_pair(wl, counts=synth.stream_counts(streams, wl.V))
    _, h = make_pair(wl, counts=synth.stream_counts(streams, wl.V))
    pinned = torch.zeros(2 * 3, dtype=torch.float64).pin_memory()
    want = []
    for t in range(3):
        for i in range(2):
            want.append(g.tensair_train_batch(i, dev(torch, streams[i][t]), t, want_loss=True)[0])
            h.tensair_train_batch(i, dev(torch, streams[i][t]), t)
            h.tensair_read_loss_async(pinned.data_ptr() + 8 * (2 * t + i))
        assert g.tensair_apply_step(t) == h.tensair_apply_step(t)
    assert h.tensair_sync() == 0
    assert pinned.tolist() == want


def test_runs_are_bit_reproducible(torch):
    wl = synth.scaled(synth.MID, V=20_000, batch=2048)
    stream = synth.token_stream(wl, 0, 4)
    counts = synth.stream_counts([stream], wl.V)
    outs = []
    for _ in range(2):
        _, g = make_pair(wl, counts=counts)
        msgs = []
        for b in range(4):
            g.tensair_train_batch(0, dev(torch, stream[b]), b)
            msgs.append(g.tensair_read_message(0, b))
        outs.append((g.tensair_read_embeddings(0, 0), g.tensair_read_embeddings(0, 1), msgs))
        g.close()
    assert np.array_equal(outs[0][0].view(np.uint32), outs[1][0].view(np.uint32))
    assert np.array_equal(outs[0][1].view(np.uint32), outs[1][1].view(np.uint32))
    for (i0, d0), (i1, d1) in zip(outs[0][2], outs[1][2]):
        assert np.array_equal(i0, i1) and np.array_equal(d0.view(np.uint32), d1.view(np.uint32))


# ------------------------------------------------------------------ many batches
def test_tiny_200_batches(torch):
    wl = synth.TINY
    stream = synth.token_stream(wl, 0)
    counts = synth.stream_counts([stream], wl.V)
    o, g = make_pair(wl, counts=counts)
    worst = 0.0
    for b in range(wl.batches):
        rc, loss_o, _ = o.train_batch(0, stream[b], b)
        assert rc == 0
        if b % 50 == 0 or b == wl.batches - 1:
            loss_g, _ = g.tensair_train_batch(0, dev(torch, stream[b]), b, want_loss=True)
            assert loss_g == pytest.approx(loss_o, rel=1e-4)
            assert np.array_equal(o.read_negatives(), g.tensair_read_negatives())
            assert np.array_equal(o.read_message(0, b)[0], g.tensair_read_message(0, b)[0])
        else:
            g.tensair_train_batch(0, dev(torch, stream[b]), b)
        if b == 0:
            compare_tables(o, g, 0, TOL_ONE)
    e = compare_tables(o, g, 0, TOL_200)
    print("tiny, 200 batches: rel err in/out", e)


def test_mid_60_batches(torch):
    wl = synth.scaled(synth.MID, batches=60)
    stream = synth.token_stream(wl, 0)
    counts = synth.stream_counts([stream], wl.V)
    o, g = make_pair(wl, counts=counts)
    for b in range(wl.batches):
        assert o.train_batch(0, stream[b], b)[0] == 0
        g.tensair_train_batch(0, dev(torch, stream[b]), b)
    assert np.array_equal(o.read_message(0, 59)[0], g.tensair_read_message(0, 59)[0])
    print("mid, 60 batches: rel err in/out", compare_tables(o, g, 0, TOL_200))


# ------------------------------------------------------------------ DASGD exchange
def _run_exchange(torch, wl, steps, drift_every=0):
    streams = synth.all_streams(wl, steps)
    counts = synth.stream_counts(streams, wl.V) if not drift_every else None
    o, g = make_pair(wl, counts=counts)
    dstreams = [dev(torch, s) for s in streams]
    for t in range(steps):
        if drift_every and t and t % drift_every == 0:
            o.update_sampler()
            g.tensair_update_sampler()
            so, sg = o.sampler(), g.tensair_read_sampler()
            assert all(np.array_equal(a, b) for a, b in zip(so, sg))
        for i in range(wl.W):
            assert o.train_batch(i, streams[i][t], t)[0] == 0
            g.tensair_train_batch(i, dstreams[i][t], t)
            if t in (0, steps - 1):
                assert np.array_equal(o.read_negatives(), g.tensair_read_negatives())
                compare_message(o, g, i, t, TOL_ONE if t == 0 else TOL_200)
        for j in range(wl.W):
            assert o.apply_messages(j, t) == g.tensair_apply_messages(j, t)
    return o, g


def test_dasgd_exchange_matches_the_oracle(torch):
    wl = synth.scaled(synth.LARGE_DASGD, V=20_000, d=48, batch=512, k=6)
    steps = 12
    o, g = _run_exchange(torch, wl, steps)
    for j in range(wl.W):
        assert np.array_equal(o.delivery_log(j), g.tensair_read_delivery_log(j))
        assert o.pending(j) == g.tensair_pending(j)
        compare_tables(o, g, j, TOL_200)
    assert o.drain() == g.tensair_drain()
    ref = None
    for j in range(wl.W):
        assert np.array_equal(o.delivery_log(j), g.tensair_read_delivery_log(j))
        assert g.tensair_pending(j) == 0
        compare_tables(o, g, j, TOL_200)
        cur = np.concatenate([g.tensair_read_embeddings(j, 0), g.tensair_read_embeddings(j, 1)])
        if ref is None:
            ref = cur
        else:   # same gradients applied everywhere, in different orders: equal up to fp32 rounding
            assert rel_err(cur, ref) <= 1e-4
    log = g.tensair_read_delivery_log(0)
    assert log[:, 4].max() > 0 and set((log[:, 2] - log[:, 0]).tolist()) == {0, 1, 2}


def test_first_step_of_the_exchange_is_within_the_one_batch_bar(torch):
    wl = synth.scaled(synth.LARGE_DASGD, V=20_000, d=300, batch=512, max_delay=0)
    o, g = _run_exchange(torch, wl, 1)
    for j in range(wl.W):
        compare_tables(o, g, j, TOL_ONE)
        assert g.tensair_read_delivery_log(j).shape[0] == wl.W - 1


def test_overwriting_an_undelivered_message_is_refused(torch):
    from paper_2211_10280_b200 import binding as B

    wl = synth.scaled(synth.TINY, V=300, d=16, W=2, max_delay=1, stream_seeds=(1, 2))
    _, g = make_pair(wl)
    toks = dev(torch, synth.token_stream(wl, 0, 1)[0])
    g.tensair_train_batch(0, toks, 0)
    g.tensair_train_batch(0, toks, 1)
    with pytest.raises(B.TensairError) as ei:
        g.tensair_train_batch(0, toks, 2)
    assert ei.value.code == B.EPENDING
    g.tensair_apply_messages(1, 1)
    g.tensair_train_batch(0, toks, 2)
    assert g.tensair_read_message(0, 0) is None and g.tensair_read_message(0, 2) is not None


def test_drift_rebuilds_the_sampler_from_running_counts(torch):
    wl = synth.scaled(synth.LARGE_DRIFT, V=5000, d=24, batch=256, W=3, k=5, drift_every=4,
                      stream_seeds=(6, 7, 8))
    o, g = _run_exchange(torch, wl, 10, drift_every=4)
    o.drain()
    g.tensair_drain()
    for j in range(wl.W):
        assert np.array_equal(o.delivery_log(j), g.tensair_read_delivery_log(j))
        compare_tables(o, g, j, TOL_200)


@pytest.mark.parametrize("V,zipf", [(2, 1.0), (3, 1.0), (1023, 1.0), (1025, 0.2), (40_000, 1.2), (1_000_000, 1.0)])
def test_alias_table_built_on_the_device_is_bit_identical(torch, V, zipf):
    """The sampler rebuilt on the device from the running counts == the oracle's table == the host builder's."""
    from paper_2211_10280_b200 import binding as B

    wl = synth.scaled(synth.TINY, V=V, d=8, window=2, k=2, batch=512, zipf_s=zipf)
    stream = synth.token_stream(wl, 0, 6)
    rng = np.random.default_rng(V)
    counts = rng.integers(1, 1000, V).astype(np.uint64) if V < 100_000 else np.ones(V, np.uint64)
    o, g = make_pair(wl, counts=counts)
    for b in range(6):
        assert o.train_batch(0, stream[b], b)[0] == 0
        g.tensair_train_batch(0, dev(torch, stream[b]), b)
    o.update_sampler()
    g.tensair_update_sampler()
    to, ao, co = o.sampler()
    tg, ag, cg = g.tensair_read_sampler()
    assert np.array_equal(co, cg)
    assert np.array_equal(to, tg) and np.array_equal(ao, ag)
    th, ah = B.tensair_build_alias_host(cg, V)
    assert np.array_equal(th, tg) and np.array_equal(ah, ag)
    B.tensair_tune("device_alias_build", 0)
    try:
        g.tensair_update_sampler()
        t2, a2, _ = g.tensair_read_sampler()
    finally:
        B.tensair_tune("device_alias_build", 1)
    assert np.array_equal(t2, tg) and np.array_equal(a2, ag)
    # and the draws of the next batch follow the new table on both sides
    toks = synth.token_stream(wl, 0, 7)[6]
    assert o.train_batch(0, toks, 6)[0] == 0
    g.tensair_train_batch(0, dev(torch, toks), 6)
    assert np.array_equal(o.read_negatives(), g.tensair_read_negatives())


def test_alias_table_of_extreme_counts_on_the_device(torch):
    V = 5000
    wl = synth.scaled(synth.TINY, V=V, d=8, window=2, k=2, batch=64)
    rng = np.random.default_rng(1)
    for counts in (rng.integers(1, 1 << 62, V, dtype=np.uint64), np.full(V, 7, np.uint64),
                   np.concatenate([np.ones(V - 1, np.uint64), np.array([10 ** 15], np.uint64)]),
                   np.uint64(16) ** rng.integers(0, 8, V).astype(np.uint64)):
        o, g = make_pair(wl, counts=counts)
        o.update_sampler()
        g.tensair_update_sampler()
        to, ao, _ = o.sampler()
        tg, ag, _ = g.tensair_read_sampler()
        assert np.array_equal(to, tg) and np.array_equal(ao, ag)


# ------------------------------------------------------------------ routed mini-batches (hash partition by centre word)
def _routed_step(torch, o, g, wl, toks, b, tol):
    """One shared batch through every replica of both sides, compared piece by piece; returns the GPU losses."""
    from paper_2211_10280_b200 import binding as B

    t_dev = dev(torch, toks)
    losses = []
    for r in range(wl.W):
        rc, loss_o, nrows_o = o.train_batch_routed(r, toks, b)
        assert rc == 0
        loss_g, info = g.tensair_train_batch_routed(r, t_dev, b, want_loss=True, want_info=True)
        assert info.n_rows == nrows_o and info.n_pairs == synth.n_pairs(len(toks), wl.window)
        assert loss_g == pytest.approx(loss_o, rel=1e-9, abs=1e-12)
        losses.append(loss_g)
        no, go = o.read_negatives(), o.read_g()
        own = no[:, 0] != 0xFFFFFFFF if no.size else np.zeros(0, bool)
        centre_owner = np.array([B.tensair_route(wl.seed, wl.W, int(x)) for x in toks])
        assert info.n_in_rows == len(set(toks[centre_owner == r].tolist()))
        if own.any():
            assert np.array_equal(g.tensair_read_negatives()[own], no[own])
            gg = g.tensair_read_scalars()[own]
            assert np.array_equal(go[own] == 0.0, gg == 0.0) and np.max(np.abs(go[own] - gg)) <= 1e-9
        if nrows_o:
            compare_message(o, g, r, b, tol)
        else:
            assert g.tensair_read_message(r, b)[0].size == 0
    for r in range(wl.W):
        assert o.apply_messages(r, b) == g.tensair_apply_messages(r, b)
    return losses


@pytest.mark.parametrize("W,reduction", [(1, 1), (2, 0), (4, 1), (8, 1)])
def test_routed_minibatch_matches_the_oracle(torch, W, reduction):
    wl = synth.scaled(synth.LARGE_DASGD, V=3000, d=36, batch=700, k=6, W=W, max_delay=1, reduction=reduction,
                      lr=0.025 if reduction else 0.002, stream_seeds=tuple(range(W)))
    stream = synth.token_stream(wl, 0, 3)
    t_in, t_out = synth.random_tables(wl.V, wl.d, 5, scale=0.3)
    o, g = make_pair(wl, counts=synth.stream_counts([stream], wl.V), init_in=t_in, init_out=t_out)
    for b in range(3):
        _routed_step(torch, o, g, wl, stream[b], b, TOL_ONE if b == 0 else TOL_200)
    assert o.drain() == g.tensair_drain()
    for r in range(W):
        assert np.array_equal(o.delivery_log(r), g.tensair_read_delivery_log(r))
        compare_tables(o, g, r, TOL_200)
    assert np.array_equal(o.sampler()[2], g.tensair_read_sampler()[2])


def test_routed_parts_add_up_to_the_single_model_step(torch):
    # the property that holds at any size: W routed parts of a batch == one model's step on the batch
    wl = synth.scaled(synth.LARGE_DASGD, V=40_000, d=64, batch=4096, k=8, W=4, max_delay=0)
    stream = synth.token_stream(wl, 0, 1)
    counts = synth.stream_counts([stream], wl.V)
    t_in, t_out = synth.random_tables(wl.V, wl.d, 6, scale=0.2)
    _, many = make_pair(wl, counts=counts, init_in=t_in, init_out=t_out)
    _, solo = make_pair(synth.scaled(wl, W=1), counts=counts, init_in=t_in, init_out=t_out)
    t_dev = dev(torch, stream[0])
    loss_solo, _ = solo.tensair_train_batch(0, t_dev, 0, want_loss=True)
    ids_solo, delta_solo = solo.tensair_read_message(0, 0)
    summed = np.zeros((2 * wl.V, wl.d))
    total, n_in = 0.0, 0
    for r in range(wl.W):
        loss_r, info = many.tensair_train_batch_routed(r, t_dev, 0, want_loss=True, want_info=True)
        total += loss_r
        n_in += info.n_in_rows
        ids_r, delta_r = many.tensair_read_message(r, 0)
        summed[ids_r] += delta_r
    assert total == pytest.approx(loss_solo, rel=1e-12)
    assert n_in == int((ids_solo < wl.V).sum())                   # input rows: a partition of the single model's
    assert set(np.flatnonzero(np.abs(summed).sum(axis=1) > 0).tolist()) <= set(ids_solo.tolist())
    # each part is rounded to fp32 on its own and parts of opposite sign cancel: a few fp32 roundings of the
    # largest part, measured against a sum that can be much smaller
    assert rel_err(summed[ids_solo], delta_solo) <= 1e-4
    for r in range(wl.W):
        assert many.tensair_apply_messages(r, 0) == wl.W - 1
    for r in range(wl.W):
        for which in (0, 1):
            assert rel_err(many.tensair_read_embeddings(r, which), solo.tensair_read_embeddings(0, which)) <= 1e-6


def test_routed_batch_of_one_word_belongs_to_one_replica(torch):
    from paper_2211_10280_b200 import binding as B

    wl = synth.scaled(synth.TINY, V=60, d=16, window=2, k=3, batch=80, W=3, max_delay=0, reduction=1,
                      stream_seeds=(1, 2, 3))
    toks = np.full(wl.batch, 11, np.int32)
    t_in, t_out = synth.random_tables(wl.V, wl.d, 2, scale=0.3)
    o, g = make_pair(wl, init_in=t_in, init_out=t_out)
    _routed_step(torch, o, g, wl, toks, 0, TOL_ONE)
    owner = B.tensair_route(wl.seed, wl.W, 11)
    for r in range(wl.W):
        ids, _ = g.tensair_read_message(r, 0)
        assert (ids.size > 0) == (r == owner)
        compare_tables(o, g, r, TOL_ONE)


# ------------------------------------------------------------------ full size, the benchmark's configuration
def test_full_size_large_dasgd_two_steps(torch):
    """V = 1M, d = 300, batch 8192, k = 15, W = 4, delay <= 2: the whole first two steps against the oracle."""
    wl = synth.LARGE_DASGD
    steps = 2
    streams = synth.all_streams(wl, steps)
    counts = synth.stream_counts(synth.all_streams(wl, 8), wl.V)
    o, g = make_pair(wl, counts=counts)
    dstreams = [dev(torch, s) for s in streams]
    rng = np.random.default_rng(0)
    for t in range(steps):
        for i in range(wl.W):
            rc, loss_o, nrows = o.train_batch(i, streams[i][t], t)
            assert rc == 0
            loss_g, info = g.tensair_train_batch(i, dstreams[i][t], t, want_loss=True, want_info=True)
            assert info.n_rows == nrows and info.n_pairs == 81_890
            assert loss_g == pytest.approx(loss_o, rel=1e-5)
            assert np.array_equal(o.read_negatives(), g.tensair_read_negatives())
            compare_message(o, g, i, t, TOL_ONE if t == 0 else 1e-4)
        for j in range(wl.W):
            assert o.apply_messages(j, t) == g.tensair_apply_messages(j, t)
    for j in range(wl.W):
        assert np.array_equal(o.delivery_log(j), g.tensair_read_delivery_log(j))
        # hot rows (most contributions) plus random rows
        rows = np.unique(np.concatenate([np.arange(2000), rng.integers(0, wl.V, 20000)]))
        for which in (0, 1):
            want = o.read_embeddings(j, which)
            got = g.tensair_read_embeddings(j, which)
            assert rel_err(got[rows], want[rows]) <= 1e-4
            assert rel_err(got, want) <= 1e-4


# ------------------------------------------------------------------ drift metric
def test_cosine_difference_of_a_snapshot_matches_the_oracle(torch):
    import oracle as orc

    wl = synth.scaled(synth.TINY, V=60_000, d=300, batches=6)
    stream = synth.token_stream(wl, 0)
    t_in, t_out = synth.random_tables(wl.V, wl.d, 12, scale=0.1)
    _, g = make_pair(wl, counts=synth.stream_counts([stream], wl.V), init_in=t_in, init_out=t_out)
    snaps = [g.tensair_snapshot_rows(0, which) for which in (0, 1)]
    assert np.array_equal(snaps[0].cpu().numpy(), t_in) and np.array_equal(snaps[1].cpu().numpy(), t_out)
    for b in range(6):
        g.tensair_train_batch(0, dev(torch, stream[b]), b)
    for which, before in ((0, t_in), (1, t_out)):
        got = g.tensair_cosine_difference(0, which, snaps[which]).cpu().numpy()
        want = orc.cosine_difference(g.tensair_read_embeddings(0, which), before)
        np.testing.assert_allclose(got, want, rtol=0, atol=2e-7)
        assert got.max() > 1e-4 and (np.abs(got) < 1e-15).sum() > 0          # touched rows moved, untouched rows did not
    part = g.tensair_snapshot_rows(0, 1, row0=100, nrows=50)
    assert np.array_equal(part.cpu().numpy(), g.tensair_read_embeddings(0, 1, 100, 50))
    assert np.abs(g.tensair_cosine_difference(0, 1, part, row0=100).cpu().numpy()).max() < 1e-15


# ------------------------------------------------------------------ launch variants give the same bits
@pytest.mark.parametrize("n,k", [(1, 1), (5, 9), (255, 4), (257, 257), (70_001, 1), (70_001, 1000), (70_001, 4096),
                                 (1_000_000, 100)])
def test_most_drifted_rows_are_bit_exact(torch, n, k):
    import oracle

    rng = np.random.default_rng(n + k)
    wl = synth.scaled(synth.TINY, V=50, d=8)
    _, g = make_pair(wl)
    cases = [rng.standard_normal(n).astype(np.float32),                       # distinct values
             (rng.integers(0, 5, n) * 0.5).astype(np.float32),                # few values, long runs of ties
             np.zeros(n, np.float32)]                                         # all equal: the first k rows
    special = rng.standard_normal(n).astype(np.float32)
    special[rng.integers(0, n, 6)] = [np.inf, -np.inf, np.nan, -0.0, 0.0, 2.0]
    cases.append(special)
    for x in cases:
        want_ids, want_vals = oracle.top_drifted(x, k)
        ids, vals = g.tensair_top_drifted(torch.from_numpy(x).cuda(), k)
        assert ids.shape[0] == min(n, k)
        assert np.array_equal(ids.cpu().numpy().view(np.uint32), want_ids)
        assert np.array_equal(vals.cpu().numpy().view(np.uint32), want_vals.view(np.uint32))


def test_most_drifted_rows_of_a_trained_table(torch):
    import oracle

    wl = synth.scaled(synth.LARGE_DRIFT, V=4000, d=32, batch=256, W=1, k=5, max_delay=0, stream_seeds=(3,))
    stream = synth.token_stream(wl, 0, 8)
    o, g = make_pair(wl, counts=synth.stream_counts([stream], wl.V))
    snap = g.tensair_snapshot_rows(0, 0)
    for b in range(8):
        g.tensair_train_batch(0, dev(torch, stream[b]), b)
    diff = g.tensair_cosine_difference(0, 0, snap)
    ids, vals = g.tensair_top_drifted(diff, 25)
    want_ids, want_vals = oracle.top_drifted(diff.cpu().numpy(), 25)
    assert np.array_equal(ids.cpu().numpy().view(np.uint32), want_ids)
    assert np.array_equal(vals.cpu().numpy(), want_vals)
    assert vals[0] > 0 and set(want_ids.tolist()) <= set(np.unique(stream).tolist())   # only trained rows move
    with pytest.raises(Exception):
        g.tensair_top_drifted(diff, 4097)


def test_fused_and_one_by_one_application_are_bit_identical(torch):
    from paper_2211_10280_b200 import binding as B

    wl = synth.scaled(synth.LARGE_DRIFT, V=30_000, d=40, batch=1024, W=5, k=6, drift_every=0,
                      stream_seeds=(6, 7, 8, 9, 10))
    streams = synth.all_streams(wl, 7)
    counts = synth.stream_counts(streams, wl.V)
    outs = []
    try:
        for fuse in (1, 0):
            B.tensair_tune("fuse_apply", fuse)
            _, g = make_pair(wl, counts=counts)
            for t in range(7):
                for i in range(wl.W):
                    g.tensair_train_batch(i, dev(torch, streams[i][t]), t)
                for j in range(wl.W):
                    g.tensair_apply_messages(j, t)
            g.tensair_drain()
            outs.append([g.tensair_read_embeddings(j, which) for j in range(wl.W) for which in (0, 1)])
            g.close()
    finally:
        B.tensair_tune("fuse_apply", 1)
    for a, b in zip(*outs):
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


@pytest.mark.parametrize("W,d,max_delay", [(5, 40, 2), (8, 300, 3), (2, 8, 0)])
def test_one_pass_for_all_receivers_equals_the_per_receiver_calls(torch, W, d, max_delay):
    """tensair_apply_step against tensair_apply_messages per replica: tables and delivery logs bit for bit, and
    both against the oracle's delivery order."""
    wl = synth.scaled(synth.LARGE_DRIFT, V=30_000, d=d, batch=1024, W=W, k=6, drift_every=0, max_delay=max_delay,
                      stream_seeds=tuple(range(30, 30 + W)))
    streams = synth.all_streams(wl, 7)
    counts = synth.stream_counts(streams, wl.V)
    o, one_pass = make_pair(wl, counts=counts)
    _, per_receiver = make_pair(wl, counts=counts)
    for t in range(7):
        for i in range(wl.W):
            assert o.train_batch(i, streams[i][t], t)[0] == 0
            one_pass.tensair_train_batch(i, dev(torch, streams[i][t]), t)
            per_receiver.tensair_train_batch(i, dev(torch, streams[i][t]), t)
        n = sum(per_receiver.tensair_apply_messages(j, t) for j in range(wl.W))
        assert one_pass.tensair_apply_step(t) == n == sum(o.apply_messages(j, t) for j in range(wl.W))
        assert one_pass.tensair_apply_step(t) == 0          # a second call for the step applies nothing
    assert one_pass.tensair_drain() == per_receiver.tensair_drain() == o.drain()
    for j in range(wl.W):
        log = one_pass.tensair_read_delivery_log(j)
        assert np.array_equal(log, per_receiver.tensair_read_delivery_log(j)) and np.array_equal(log, o.delivery_log(j))
        for which in (0, 1):
            a, b = one_pass.tensair_read_embeddings(j, which), per_receiver.tensair_read_embeddings(j, which)
            assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), (j, which)
        compare_tables(o, one_pass, j, TOL_200)


def test_full_size_drift_workload_with_sampler_rebuild(torch):
    """V = 1M, d = 300, batch 16384, k = 15, W = 8, delay <= 2, Zipf 1.1 with a permuted vocabulary: two steps,
    the sampler rebuilt from the running counts in between, everything against the oracle."""
    wl = synth.scaled(synth.LARGE_DRIFT, drift_every=1)
    steps = 2
    streams = synth.all_streams(wl, steps)
    o, g = make_pair(wl)
    dstreams = [dev(torch, s) for s in streams]
    for t in range(steps):
        if t:
            o.update_sampler()
            g.tensair_update_sampler()
            assert all(np.array_equal(a, b) for a, b in zip(o.sampler(), g.tensair_read_sampler()))
        for i in range(wl.W):
            rc, loss_o, nrows = o.train_batch(i, streams[i][t], t)
            assert rc == 0
            loss_g, info = g.tensair_train_batch(i, dstreams[i][t], t, want_loss=True, want_info=True)
            assert info.n_rows == nrows and info.n_pairs == 163_810
            assert loss_g == pytest.approx(loss_o, rel=1e-5)
            if i in (0, wl.W - 1):
                assert np.array_equal(o.read_negatives(), g.tensair_read_negatives())
                compare_message(o, g, i, t, TOL_ONE if t == 0 else 1e-4)
        for j in range(wl.W):
            assert o.apply_messages(j, t) == g.tensair_apply_messages(j, t)
    for j in (0, 3, wl.W - 1):
        assert np.array_equal(o.delivery_log(j), g.tensair_read_delivery_log(j))
        for which in (0, 1):
            assert rel_err(g.tensair_read_embeddings(j, which), o.read_embeddings(j, which)) <= 1e-4


# ------------------------------------------------------------------ maxGradBuffer > 1
@pytest.mark.parametrize("m", [2, 3])
def test_buffered_gradients_are_sent_every_mth_batch(torch, m):
    """Algorithm 1 with maxGradBuffer = m: union of rows, summed deltas, m times fewer messages."""
    wl = synth.scaled(synth.LARGE_DASGD, V=30_000, d=44, batch=512, k=6, W=3, stream_seeds=(2, 3, 4))
    steps = 11
    streams = synth.all_streams(wl, steps)
    t_in, t_out = synth.random_tables(wl.V, wl.d, 21, scale=0.2)
    o, g = make_pair(wl, counts=synth.stream_counts(streams, wl.V), init_in=t_in, init_out=t_out, max_grad_buffer=m)
    applied = 0
    for t in range(steps):
        for i in range(wl.W):
            assert o.train_batch(i, streams[i][t], t)[0] == 0
            g.tensair_train_batch(i, dev(torch, streams[i][t]), t)
            om, gm = o.read_message(i, t), g.tensair_read_message(i, t)
            assert (om is None) == (gm is None) == (t % m != m - 1)
            if om is not None:
                assert np.array_equal(om[0], gm[0])
                assert rel_err(gm[1], om[1]) <= TOL_200
        for j in range(wl.W):
            n = o.apply_messages(j, t)
            assert n == g.tensair_apply_messages(j, t)
            applied += n
    assert o.drain() == g.tensair_drain()
    sends = steps // m
    for j in range(wl.W):
        log = g.tensair_read_delivery_log(j)
        assert np.array_equal(o.delivery_log(j), log) and log.shape[0] == sends * (wl.W - 1)
        assert set((log[:, 0] % m).tolist()) == {m - 1}
        compare_tables(o, g, j, TOL_200)


def test_merged_message_larger_than_any_one_batch_message(torch):
    """maxGradBuffer = 8 with few contributions per batch and a large vocabulary: the union of the 8 buffered
    messages has several times the rows any single batch can touch, so the send slot must be sized for the union."""
    m = 8
    wl = synth.scaled(synth.LARGE_DASGD, V=200_000, d=16, window=2, batch=64, k=3, W=2, stream_seeds=(2, 3),
                      max_delay=1, zipf_s=0.2)
    one_batch = wl.batch + wl.pairs_per_batch * (wl.k + 1)
    steps = 2 * m
    streams = synth.all_streams(wl, steps)
    t_in, t_out = synth.random_tables(wl.V, wl.d, 22, scale=0.2)
    o, g = make_pair(wl, counts=synth.stream_counts(streams, wl.V), init_in=t_in, init_out=t_out, max_grad_buffer=m)
    assert g.sizes.max_rows == m * one_batch
    largest = 0
    for t in range(steps):
        for i in range(wl.W):
            assert o.train_batch(i, streams[i][t], t)[0] == 0
            g.tensair_train_batch(i, dev(torch, streams[i][t]), t)
            om, gm = o.read_message(i, t), g.tensair_read_message(i, t)
            assert (om is None) == (gm is None) == (t % m != m - 1)
            if om is not None:
                largest = max(largest, om[0].size)
                assert np.array_equal(om[0], gm[0])
                assert rel_err(gm[1], om[1]) <= TOL_200
        for j in range(wl.W):
            assert o.apply_messages(j, t) == g.tensair_apply_messages(j, t)
    assert largest > 3 * one_batch, (largest, one_batch)      # the case the one-batch bound would have overflowed
    assert o.drain() == g.tensair_drain()
    assert g.tensair_sync() == 0
    for j in range(wl.W):
        compare_tables(o, g, j, TOL_200)


def test_a_wait_that_ran_out_is_not_reported_as_a_bad_token(torch):
    """The device error word is raised from the host, as a kernel whose bounded wait gave up would raise it
    (no GPU is made to misbehave): every cause has its own code, and reading the word clears it."""
    from paper_2211_10280_b200 import binding as B

    wl = synth.scaled(synth.TINY, V=500, d=8, batch=64)
    g = B.Context(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch)
    assert g.tensair_sync() == B.OK
    g.tensair_raise_error_flags(2)
    assert g.tensair_sync() == B.ETIMEOUT and "wait" in g.tensair_last_error()
    assert g.tensair_sync() == B.OK
    g.tensair_raise_error_flags(1)
    assert g.tensair_sync() == B.EBADTOKEN and "token" in g.tensair_last_error()
    g.tensair_raise_error_flags(1)
    g.tensair_raise_error_flags(2)
    assert g.tensair_sync() == B.ETIMEOUT          # the graver of the two; the text names both
    assert "token" in g.tensair_last_error() and "wait" in g.tensair_last_error()
    g.tensair_raise_error_flags(8)
    assert g.tensair_sync() == B.EBOUNDS
    # a raised word drops the batches that follow until it has been read, like a bad token does
    before = g.tensair_read_embeddings(0, 1)
    g.tensair_raise_error_flags(2)
    g.tensair_train_batch(0, dev(torch, synth.token_stream(wl, 0, 1)[0]), 0)
    assert g.tensair_sync() == B.ETIMEOUT
    assert np.array_equal(g.tensair_read_embeddings(0, 1), before)


def test_largest_sweep_batch_matches_the_oracle(torch):
    """One batch of the throughput sweep's largest shape (V = 1M, batch 65,536, k = 15, window 5) at d = 64:
    10.5 M contributions, more than 2,500 sort tiles, hot rows with tens of thousands of contributions (hundreds to
    thousands of 64-term chunks each).  Negatives and message ids bit-exact, scalars, deltas and tables within the
    one-batch bar."""
    wl = synth.sweep_point(64, 65536, 15)
    stream = synth.token_stream(wl, 0, 1)
    counts = synth.stream_counts([stream], wl.V)
    t_in, t_out = synth.random_tables(wl.V, wl.d, 23, scale=2.0 / math.sqrt(wl.d))
    o, g = make_pair(wl, counts=counts, init_in=t_in, init_out=t_out)
    rc, loss_o, nrows_o = o.train_batch(0, stream[0], 0)
    assert rc == 0
    loss_g, info = g.tensair_train_batch(0, dev(torch, stream[0]), 0, want_loss=True, want_info=True)
    assert info.n_pairs == wl.pairs_per_batch == 655_330
    assert 2 * wl.batch + info.n_pairs * (wl.k + 1) > 2500 * 4096          # sort tiles of 4,096 items
    assert info.n_rows == nrows_o
    no, ng = o.read_negatives(), g.tensair_read_negatives()
    assert np.array_equal(no, ng)
    # contributions per output row: the unmasked negative draws on it plus the pairs whose context word it is
    toks = stream[0].astype(np.int64)
    pos = np.arange(wl.batch)
    as_context = np.minimum(pos, wl.window) + np.minimum(wl.batch - 1 - pos, wl.window)
    per_row = np.bincount(toks, weights=as_context, minlength=wl.V) + np.bincount(no.ravel(), minlength=wl.V)
    assert per_row.max() > 64 * 500, per_row.max()                           # a row of more than 500 chunks
    assert (per_row > 64).sum() > 500                                        # and hundreds of rows on the chunked path
    go, gg = o.read_g(), g.tensair_read_scalars()
    assert np.max(np.abs(go - gg)) <= 1e-13
    assert loss_g == pytest.approx(loss_o, rel=1e-12)
    compare_message(o, g, 0, 0, TOL_ONE)
    compare_tables(o, g, 0, TOL_ONE)


def test_subnormal_rows_and_deltas_are_added_like_the_oracle_adds_them(torch):
    """Table entries and deltas around the smallest normal fp32 (2^-126): the additions that apply a message (the
    local application of the output rows inside the row-sum kernel, the input rows, and the remote application) must
    keep subnormal inputs and results as IEEE arithmetic does - the oracle's `row + delta` in fp32 - bit for bit."""
    wl = synth.scaled(synth.TINY, V=300, d=20, window=2, k=4, batch=200, W=2, stream_seeds=(0, 1), lr=1.0, max_delay=0)
    streams = synth.all_streams(wl, 1)
    t_in, t_out = synth.random_tables(wl.V, wl.d, 29, scale=1.0)
    tiny = np.float32(2.0 ** -125)
    t_in, t_out = (t_in * tiny).astype(np.float32), (t_out * tiny).astype(np.float32)
    sub = np.float32(2.0 ** -126)
    assert (np.abs(t_out[t_out != 0]) < sub).mean() > 0.3 and (np.abs(t_out) >= sub).mean() > 0.3
    o, g = make_pair(wl, counts=synth.stream_counts(streams, wl.V), init_in=t_in, init_out=t_out)
    for i in range(wl.W):
        assert o.train_batch(i, streams[i][0], 0)[0] == 0
        g.tensair_train_batch(i, dev(torch, streams[i][0]), 0)
        ids_o, delta_o = o.read_message(i, 0)
        ids_g, delta_g = g.tensair_read_message(i, 0)
        assert np.array_equal(ids_o, ids_g)
        # every dot product is ~1e-74, every sigmoid 1/2 to the last bit: a delta is one rounding of an exact sum
        assert np.array_equal(delta_o.view(np.uint32), delta_g.view(np.uint32))
        small = np.abs(delta_o[delta_o != 0]) < sub
        assert small.any() and not small.all()
    for i in range(wl.W):                                # local application, output and input rows
        for which in (0, 1):
            assert np.array_equal(o.read_embeddings(i, which).view(np.uint32),
                                  g.tensair_read_embeddings(i, which).view(np.uint32)), (i, which)
    for j in range(wl.W):                                # remote application
        assert o.apply_messages(j, 0) == g.tensair_apply_messages(j, 0) == 1
        for which in (0, 1):
            got = g.tensair_read_embeddings(j, which)
            assert np.array_equal(o.read_embeddings(j, which).view(np.uint32), got.view(np.uint32)), (j, which)
    assert (np.abs(got[got != 0]) < sub).any()


def test_long_parity_runner_on_a_short_drifting_run(torch):
    """tests/long_parity.py (the runner of the full-length parity runs) on a reduced drifting workload: 25 steps of
    3 replicas across two sampler rebuilds, checked every 10 steps."""
    import long_parity

    wl = synth.scaled(synth.LARGE_DRIFT, V=8000, d=40, batch=256, W=3, k=5, drift_every=10, stream_seeds=(6, 7, 8))
    res = long_parity.run(wl, steps=25, check_every=10)
    assert res["sampler_rebuilds"] == 2 and [c["step"] for c in res["checks"]] == [10, 20, 25]
    assert res["max_rel_err"] <= TOL_200 and res["after_drain"] <= TOL_200


def test_checked_build_reports_a_row_id_outside_the_table_and_skips_it(torch):
    """Only with the checked build loaded (TENSAIR_CHECKED=1): a received message that names a row past the end of
    the receiver's table (a corrupted transfer) is reported as TENSAIR_EBOUNDS and the row is left out; the rows in
    range are applied.  (The address the bad id stands for lies inside the tables buffer - in the other local
    replica's table - so even the normal build, where this test is skipped, would not touch foreign memory.)"""
    from paper_2211_10280_b200 import binding as B

    if not B.lib().tensair_checked_build():
        pytest.skip("needs the checked build: TENSAIR_CHECKED=1 with libtensair_checked.so built")
    V, d = 400, 8
    g = B.Context(V=V, d=d, window=2, k=3, batch=32, W=2, world_replicas=3, first_replica=0, max_delay=0)
    before = [[g.tensair_read_embeddings(r, w) for w in (0, 1)] for r in range(2)]
    ids, delta = g.tensair_message_buffers(2, 0)
    stride = delta.numel() // ids.numel()
    ids[:2].copy_(torch.tensor([7, 2 * V + 5], dtype=torch.int32))
    delta[:2 * stride].fill_(0.25)
    g.tensair_commit_message(2, 0, 2, 1)
    assert g.tensair_apply_messages(0, 0) == 1
    assert g.tensair_sync() == B.EBOUNDS and "outside its array" in g.tensair_last_error()
    after = [[g.tensair_read_embeddings(r, w) for w in (0, 1)] for r in range(2)]
    want = before[0][0].copy()
    want[7] += np.float32(0.25)
    assert np.array_equal(after[0][0], want) and np.array_equal(after[0][1], before[0][1])
    assert np.array_equal(after[1][0], before[1][0]) and np.array_equal(after[1][1], before[1][1])
    assert g.tensair_sync() == B.OK


@pytest.mark.parametrize("m", [1, 2])
def test_a_run_saved_in_flight_resumes_bit_for_bit(torch, m):
    """Tables and pool copied by the caller, the library's part by tensair_save_state, in the middle of a step (batches
    trained, their messages not yet applied, older messages still pending); a fresh context given all three goes on to
    compute exactly what the uninterrupted run computes - tables, messages, delivery order and staleness."""
    from paper_2211_10280_b200 import binding as B

    wl = synth.scaled(synth.LARGE_DRIFT, V=6000, d=24, batch=256, W=3, k=5, drift_every=4, stream_seeds=(6, 7, 8),
                      max_delay=2)
    steps, cut = 11, 4                              # with m = 2 every replica holds one buffered message at the cut
    streams = synth.all_streams(wl, steps)
    kw = dict(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch, W=wl.W, lr=wl.lr, max_delay=wl.max_delay,
              seed=wl.seed, reduction=wl.reduction, max_grad_buffer=m)
    a = B.Context(**kw)

    def train(ctx, t):
        if t and t % wl.drift_every == 0:
            ctx.tensair_update_sampler()
        for i in range(wl.W):
            ctx.tensair_train_batch(i, dev(torch, streams[i][t]), t)

    for t in range(cut):
        train(a, t)
        a.tensair_apply_step(t)
    train(a, cut)                                   # the cut: step `cut` trained, nothing of it applied
    assert a.tensair_sync() == B.OK
    blob = a.tensair_save_state()
    tables = [[a.tensair_read_embeddings(r, w) for w in (0, 1)] for r in range(wl.W)]
    pool = a.pool.clone()
    b = B.Context(**kw)
    b.tensair_load_state(blob)
    for r in range(wl.W):
        for w in (0, 1):
            b.tensair_write_embeddings(r, w, 0, tables[r][w])
    b.pool.copy_(pool)
    assert all(np.array_equal(x, y) for x, y in zip(a.tensair_read_sampler(), b.tensair_read_sampler()))
    for ctx in (a, b):
        ctx.tensair_apply_step(cut)
        for t in range(cut + 1, steps):
            train(ctx, t)
            ctx.tensair_apply_step(t)
        ctx.tensair_drain()
        assert ctx.tensair_sync() == B.OK
    for r in range(wl.W):
        la, lb = a.tensair_read_delivery_log(r), b.tensair_read_delivery_log(r)
        assert np.array_equal(la, lb) and la.shape[0] > 0
        for w in (0, 1):
            assert np.array_equal(a.tensair_read_embeddings(r, w).view(np.uint32), b.tensair_read_embeddings(r, w).view(np.uint32))
    # a state saved under another configuration is refused
    other = B.Context(**dict(kw, max_delay=1))
    with pytest.raises(B.TensairError) as e:
        other.tensair_load_state(blob)
    assert e.value.code == B.EINVAL
