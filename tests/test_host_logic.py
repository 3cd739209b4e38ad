"""Host-side logic of the CUDA library, checked without a GPU: exported symbols, Philox, the alias
table build, the delivery schedule and its staleness bookkeeping, workspace sizing, argument checks."""
import ctypes as C
import re
import subprocess
from pathlib import Path

import numpy as np
import pytest

import oracle
from oracle import Oracle
from paper_2211_10280_b200 import binding as B
from paper_2211_10280_b200 import build as libbuild
from paper_2211_10280_b200 import synth

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module", autouse=True)
def _built():
    libbuild.build()


def _declared():
    text = (ROOT / "include" / "tensair.h").read_text()
    return sorted(set(re.findall(r"TENSAIR_API[^;(]*?\b(tensair_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared()
    assert len(names) >= 25
    out = subprocess.check_output(["nm", "-D", "--defined-only", str(B.LIB_PATH)], text=True)
    exported = {line.split()[-1] for line in out.splitlines() if " T " in line}
    assert set(names) <= exported
    assert {n for n in exported if n.startswith("tensair_")} == set(names)
    lib = C.CDLL(str(B.LIB_PATH))
    for n in names:
        assert getattr(lib, n) is not None
    assert sorted(B.SYMBOLS) == names


def test_philox_known_answers(golden_dir):
    for line in open(golden_dir / "philox4x32_10_kat.txt"):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        assert B.tensair_philox4x32_10(w[:4], w[4:6]) == w[6:]


@pytest.mark.parametrize("V,seed", [(2, 0), (9, 1), (1000, 2), (50_000, 3)])
def test_alias_table_is_bit_identical_to_the_oracle(V, seed):
    rng = np.random.default_rng(seed)
    counts = (rng.zipf(1.2, V).astype(np.uint64) % 1_000_000) + 1
    t0, a0 = oracle.build_alias(counts)
    t1, a1 = B.tensair_build_alias_host(counts, V)
    assert np.array_equal(t0, t1) and np.array_equal(a0, a1)


@pytest.mark.parametrize("case", ["huge", "ones_and_one_big", "two_values", "powers_of_16", "V3"])
def test_alias_table_corner_cases_are_bit_identical_to_the_oracle(case):
    rng = np.random.default_rng(8)
    counts = {
        "huge": rng.integers(1, 1 << 62, 4000, dtype=np.uint64),
        "ones_and_one_big": np.concatenate([np.ones(999, np.uint64), np.array([10 ** 12], np.uint64)]),
        "two_values": rng.choice(np.array([3, 48], np.uint64), 2048),
        "powers_of_16": np.uint64(16) ** rng.integers(0, 8, 1000).astype(np.uint64),   # exact weights 8^j
        "V3": np.array([5, 5, 1], np.uint64),
    }[case]
    t0, a0 = oracle.build_alias(counts)
    t1, a1 = B.tensair_build_alias_host(counts, counts.size)
    assert np.array_equal(t0, t1) and np.array_equal(a0, a1)


def test_alias_table_of_a_zipf_stream_matches_the_oracle():
    wl = synth.scaled(synth.MID, batches=20)
    counts = synth.stream_counts([synth.token_stream(wl, 0)], wl.V)
    t0, a0 = oracle.build_alias(counts)
    t1, a1 = B.tensair_build_alias_host(counts, wl.V)
    assert np.array_equal(t0, t1) and np.array_equal(a0, a1)
    t2, a2 = B.tensair_build_alias_host(None, 77)
    assert np.all(t2 == 0xFFFFFFFF) and np.array_equal(a2, np.arange(77, dtype=np.uint32))


def test_alias_rejects_zero_counts():
    lib = B.lib()
    c = np.array([1, 0, 3], np.uint64)
    t = np.empty(3, np.uint32)
    assert lib.tensair_build_alias_host(c.ctypes.data_as(C.c_void_p), 3, t.ctypes.data_as(C.c_void_p),
                                        t.ctypes.data_as(C.c_void_p)) == B.EINVAL


def test_delay_matches_the_oracle_and_is_uniform():
    o = Oracle(V=4, d=4, window=1, k=1, batch=2, W=5, max_delay=2, seed=0xABCDEF0123)
    seen = np.zeros(3, int)
    for t in range(200):
        for i in range(5):
            for j in range(5):
                dl = B.tensair_delay(0xABCDEF0123, 2, t, i, j)
                assert dl == o.delay(t, i, j)
                seen[dl] += 1
    assert seen.min() > 0.28 * seen.sum()
    assert all(B.tensair_delay(1, 0, t, 0, 1) == 0 for t in range(20))


def test_route_matches_the_oracle():
    for W in (1, 2, 3, 4, 8):
        for seed in (0, 0xABCDEF0123):
            assert [B.tensair_route(seed, W, x) for x in range(300)] == [oracle.route(seed, W, x) for x in range(300)]
    out = C.c_uint32(0)
    assert B.lib().tensair_route(1, 0, 5, C.byref(out)) == B.EINVAL
    assert B.lib().tensair_route(1, 2, 5, None) == B.EINVAL


def _oracle_logs(W, D, T, seed, skip=()):
    o = Oracle(V=16, d=4, window=1, k=1, batch=4, W=W, max_delay=D, seed=seed)
    toks = np.array([1, 2, 3, 4], np.int32)
    for t in range(T):
        for i in range(W):
            if (i, t) not in skip:
                assert o.train_batch(i, toks, t)[0] == 0
        for j in range(W):
            o.apply_messages(j, t)
    return o


@pytest.mark.parametrize("W,D,T", [(2, 0, 5), (3, 2, 40), (4, 2, 30), (8, 2, 12), (3, 5, 300)])
def test_schedule_matches_the_oracle_log_bit_for_bit(W, D, T):
    seed = 1234 + W
    o = _oracle_logs(W, D, T, seed)
    s = B.Schedule(W, D, seed)
    got = [[] for _ in range(W)]
    for t in range(T):
        for i in range(W):
            assert s.on_train(i, t) == B.OK
        for j in range(W):
            got[j].extend(s.take_due(j, t).tolist())
    for j in range(W):
        assert s.pending(j) == o.pending(j)
    assert o.drain() == sum(s.pending(j) for j in range(W))
    for j in range(W):
        got[j].extend(s.take_due(j, 0, drain=True).tolist())
        assert got[j] == o.delivery_log(j).tolist()
        assert s.pending(j) == 0


def test_schedule_with_idle_replicas_matches_the_oracle():
    # replicas may skip steps (the mini-batch generator hands batches to whichever model it picks)
    W, D, T, seed = 3, 2, 20, 5
    skip = {(0, t) for t in range(0, T, 3)} | {(2, t) for t in range(5, 12)}
    o = _oracle_logs(W, D, T, seed, skip)
    s = B.Schedule(W, D, seed)
    got = [[] for _ in range(W)]
    for t in range(T):
        for i in range(W):
            if (i, t) not in skip:
                assert s.on_train(i, t) == B.OK
        for j in range(W):
            got[j].extend(s.take_due(j, t).tolist())
    o.drain()
    for j in range(W):
        got[j].extend(s.take_due(j, 0, drain=True).tolist())
        assert got[j] == o.delivery_log(j).tolist()


def test_schedule_refuses_to_overwrite_an_undelivered_message():
    s = B.Schedule(2, 1, 7)
    assert s.on_train(0, 0) == B.OK
    assert s.on_train(0, 1) == B.OK
    # step 2 would reuse the slot of step 0, whose message replica 1 has not taken yet
    assert s.on_train(0, 2) == B.EPENDING
    s.take_due(1, 1)
    assert s.on_train(0, 2) == B.OK
    assert s.on_train(5, 0) == B.EINVAL


def test_fig2_example_through_the_schedule(golden_dir):
    # Models 1..3 -> replicas 0..2.  Step 0: all three compute (red, blue, green); step 1: only Model 2
    # computes (yellow).  green reaches Model 2 after yellow; red reaches it after green.  With the
    # library's seeded delays that order needs delay(green -> 2) = 1 and delay(red -> 2) = 2, so search a seed.
    want = {}
    for line in open(golden_dir / "fig2_staleness.txt"):
        if not line.startswith("#") and line.strip():
            ev, _, grad, val = line.split()
            want[(ev, grad)] = int(val)
    seed = next(s for s in range(10_000)
                if B.tensair_delay(s, 2, 0, 2, 1) == 1 and B.tensair_delay(s, 2, 0, 0, 1) == 2)
    s = B.Schedule(3, 2, seed)
    for i in range(3):
        assert s.on_train(i, 0) == B.OK
    assert s.take_due(1, 0).shape[0] == 0
    assert s.on_train(1, 1) == B.OK
    green = s.take_due(1, 1).tolist()
    assert [r[1] for r in green] == [2] and green[0][4] == want[("staleness", "green")]
    red = s.take_due(1, 2).tolist()
    assert [r[1] for r in red] == [0] and red[0][4] == want[("staleness", "red")]


def test_workspace_sizes():
    cfg = B.Config(V=1_000_000, d=300, window=5, k=15, batch=8192, W=4, lr=0.025, max_grad_buffer=1,
                   max_delay=2, row_stride=0, seed=0, device=0, reduction=1)
    sz = B.tensair_workspace_bytes(cfg)
    assert sz.row_stride == 304
    assert sz.max_pairs == synth.n_pairs(8192, 5) == 81_890
    assert sz.tables_bytes == 4 * 2 * 1_000_000 * 304 * 4
    assert sz.max_rows == 8192 + 1_000_000
    assert sz.pool_bytes >= 4 * 3 * sz.max_rows * 304 * 4
    assert sz.scratch_bytes < 2 << 30


@pytest.mark.parametrize("field,value", [("V", 1), ("d", 6), ("d", 2048), ("window", 0), ("window", 17), ("k", 0),
                                         ("batch", 0), ("W", 0), ("max_grad_buffer", 0), ("max_grad_buffer", 9), ("row_stride", 2),
                                         ("reduction", 2)])
def test_unsupported_configurations_are_rejected(field, value):
    kw = dict(V=100, d=8, window=2, k=3, batch=16, W=1, lr=0.025, max_grad_buffer=1, max_delay=0, row_stride=0,
              seed=0, device=0, reduction=0)
    kw[field] = value
    out = B.Sizes()
    assert B.lib().tensair_workspace_bytes(C.byref(B.Config(**kw)), C.byref(out)) == B.EINVAL


def test_null_arguments_are_rejected_not_dereferenced():
    lib = B.lib()
    assert lib.tensair_workspace_bytes(None, None) == B.EINVAL
    assert lib.tensair_train_batch(None, 0, None, 0, 0, None, None) == B.EINVAL
    assert lib.tensair_apply_messages(None, 0, 0, None) == B.EINVAL
    assert lib.tensair_read_embeddings(None, 0, 0, 0, 0, None) == B.EINVAL
    assert lib.tensair_kernel_launches(None) == 0
    assert lib.tensair_strerror(B.EPENDING).decode().startswith("message slot")
    lib.tensair_destroy(None)


def test_device_error_word_is_decoded_bit_by_bit():
    # bit 0 bad token, bit 1 a bounded wait that ran out, bits 2 and 3 an index or a merged message out of bounds:
    # each has its own code, and the gravest of several wins
    assert B.tensair_error_of_flags(0) == B.OK
    assert B.tensair_error_of_flags(1) == B.EBADTOKEN
    assert B.tensair_error_of_flags(2) == B.ETIMEOUT
    assert B.tensair_error_of_flags(4) == B.EBOUNDS
    assert B.tensair_error_of_flags(8) == B.EBOUNDS
    assert B.tensair_error_of_flags(1 | 2) == B.ETIMEOUT
    assert B.tensair_error_of_flags(1 | 2 | 4) == B.EBOUNDS
    assert len({B.EBADTOKEN, B.ETIMEOUT, B.EBOUNDS, B.ECUDA}) == 4
    assert "wait" in B.strerror(B.ETIMEOUT) and "index" in B.strerror(B.EBOUNDS)


@pytest.mark.parametrize("m", [1, 2, 8])
def test_message_slots_hold_the_union_of_the_buffered_messages(m):
    # batch 256, window 5, k 5: 15,180 contributions and 256 centre words per batch, far below V, so the union of
    # m buffered messages can have m times the rows of one
    cfg = B.Config(V=1_000_000, d=64, window=5, k=5, batch=256, W=1, lr=0.025, max_grad_buffer=m,
                   max_delay=0, row_stride=0, seed=0, device=0, reduction=1)
    sz = B.tensair_workspace_bytes(cfg)
    contrib = synth.n_pairs(256, 5) * 6
    assert sz.max_rows == m * 256 + m * contrib
    slots = 1 + (m if m > 1 else 0)
    assert sz.pool_bytes >= slots * sz.max_rows * (64 * 4 + 4)
    # capped by the tables: a message cannot have more rows than the model
    big = B.Config(V=1000, d=64, window=5, k=5, batch=256, W=1, lr=0.025, max_grad_buffer=m,
                   max_delay=0, row_stride=0, seed=0, device=0, reduction=1)
    assert B.tensair_workspace_bytes(big).max_rows == min(m * 256, 1000) + 1000


def test_sharded_job_with_buffered_gradients_is_refused():
    cfg = B.Config(V=100, d=8, window=2, k=3, batch=16, W=1, lr=0.025, max_grad_buffer=2, max_delay=0, row_stride=0,
                   seed=0, device=0, reduction=0)
    sz = B.tensair_workspace_bytes_sharded(cfg, 2)
    # the refusal comes before any buffer or device is touched: fake, aligned, large-enough buffers will do
    bufs = B.Buffers(256, sz.tables_bytes, 256, sz.pool_bytes, 256, sz.scratch_bytes, None)
    h = C.c_void_p()
    assert B.lib().tensair_init_sharded(C.byref(cfg), C.byref(bufs), None, None, None, 0, 2, C.byref(h)) == B.EINVAL
    assert not h.value


def test_schedule_saved_and_loaded_continues_as_if_never_interrupted():
    W, D, seed = 4, 2, 5
    a = B.Schedule(W, D, seed)
    for t in range(70):                       # past the point where fully applied gradients are trimmed from the sets
        for g in range(W):
            assert a.on_train(g, t) == B.OK
        for g in range(W):
            a.take_due(g, t)
    for g in range(W):
        assert a.on_train(g, 70) == B.OK      # saved with the messages of step 70 computed and none of them applied
    blob = a.save()
    b = B.Schedule(W, D, seed)
    assert b.load(blob) == B.OK
    assert [b.pending(g) for g in range(W)] == [a.pending(g) for g in range(W)] and sum(a.pending(g) for g in range(W)) > 0
    for t in range(70, 90):
        if t > 70:
            for g in range(W):
                assert a.on_train(g, t) == b.on_train(g, t) == B.OK
        for g in range(W):
            assert np.array_equal(a.take_due(g, t), b.take_due(g, t))      # order, due steps and staleness
    for g in range(W):
        assert np.array_equal(a.take_due(g, 0, True), b.take_due(g, 0, True))
    # a schedule of another shape, or damaged bytes, are refused and change nothing
    assert B.Schedule(W, D + 1, seed).load(blob) == B.EINVAL
    assert B.Schedule(W, D, seed + 1).load(blob) == B.EINVAL
    c = B.Schedule(W, D, seed)
    assert c.load(blob[:-8]) == B.EINVAL and c.load(blob + b"\0" * 8) == B.EINVAL
    assert c.on_train(0, 0) == B.OK           # the refused loads left it untouched
    for at in range(48, len(blob) - 8, 8):      # any one field overwritten: refused or accepted, never a crash
        assert B.Schedule(W, D, seed).load(blob[:at] + b"\xff" * 8 + blob[at + 8:]) in (B.EINVAL, B.OK)
