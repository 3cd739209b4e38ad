"""tensair_train_batch_static: the mini-batch step for callers that must not allocate device memory.

Such a caller (a plug-in living inside a host application's fixed memory plan, a service thread kept out
of the allocator) cannot size and provide per-batch scratch; the entry point takes it from a fixed array
inside the library.  The check: through the C ABI, on the same seeded inputs, two calls in a row must
give what tensair_train_batch gives - same loss, same message rows, deltas and tables within the
one-batch parity tolerance (they are in fact bit-identical) - and what the CPU oracle gives for the same
batches; and a call that is not the first on its device must leave the device's free memory exactly as
it found it.  This file sorts last on purpose, so that a run that stops at the first failure has already
run every other test; it also passes on its own.
"""
import numpy as np
import pytest

from parity_utils import compare_message, compare_tables, rel_err
from paper_2211_10280_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-5


def _context(wl, counts, t_in, t_out):
    from paper_2211_10280_b200 import binding as B

    return B.Context(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch, W=wl.W, lr=wl.lr,
                     max_delay=wl.max_delay, seed=wl.seed, counts=counts, init_in=t_in, init_out=t_out,
                     reduction=wl.reduction)


def test_static_scratch_entry_point_matches_train_batch_on_two_calls_in_a_row():
    import torch

    assert torch.cuda.is_available(), "this test needs a CUDA device"
    wl = synth.scaled(synth.MID, V=20_000, d=64, batch=1024, batches=2)
    stream = synth.token_stream(wl, 0)
    counts = synth.stream_counts([stream], wl.V)
    t_in, t_out = synth.random_tables(wl.V, wl.d, 31, scale=0.25)
    from oracle import Oracle

    ref, new = _context(wl, counts, t_in, t_out), _context(wl, counts, t_in, t_out)
    orc = Oracle(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch, W=wl.W, lr=wl.lr, max_delay=wl.max_delay,
                 seed=wl.seed, counts=counts, init_in=t_in, init_out=t_out, reduction=wl.reduction)
    for b in range(2):
        toks = torch.from_numpy(stream[b]).cuda()
        torch.cuda.synchronize()
        loss_ref, info_ref = ref.tensair_train_batch(0, toks, b, want_loss=True, want_info=True)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        loss_new, info_new = new.tensair_train_batch_static(0, toks, b, want_loss=True, want_info=True)
        torch.cuda.synchronize()
        if b > 0:       # the first call on a device may make the driver load the module that holds the array
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
        rc, loss_orc, rows_orc = orc.train_batch(0, stream[b], b)
        assert rc == 0 and info_new.n_rows == rows_orc
        assert loss_new == pytest.approx(loss_orc, rel=1e-12)
        assert np.array_equal(new.tensair_read_negatives(), orc.read_negatives())
        assert np.max(np.abs(new.tensair_read_scalars() - orc.read_g())) <= 1e-13
        compare_message(orc, new, 0, b, TOL)
        compare_tables(orc, new, 0, (b + 1) * TOL)
        assert (info_new.n_rows, info_new.n_in_rows, info_new.n_pairs) == (info_ref.n_rows, info_ref.n_in_rows, info_ref.n_pairs)
        assert loss_new == pytest.approx(loss_ref, rel=1e-12)
        assert np.array_equal(new.tensair_read_negatives(), ref.tensair_read_negatives())
        ids_ref, delta_ref = ref.tensair_read_message(0, b)
        ids_new, delta_new = new.tensair_read_message(0, b)
        assert np.array_equal(ids_new, ids_ref)
        assert rel_err(delta_new, delta_ref) <= TOL
        for which in (0, 1):
            assert rel_err(new.tensair_read_embeddings(0, which), ref.tensair_read_embeddings(0, which)) <= TOL
    # the array keeps the previous call's contents: a shorter batch after a longer one must not see them
    short = torch.from_numpy(stream[0][:37].copy()).cuda()
    l_ref, _ = ref.tensair_train_batch(0, short, 2, want_loss=True)
    l_new, _ = new.tensair_train_batch_static(0, short, 2, want_loss=True)
    assert l_new == pytest.approx(l_ref, rel=1e-12)
    assert np.array_equal(new.tensair_read_message(0, 2)[0], ref.tensair_read_message(0, 2)[0])
    assert rel_err(new.tensair_read_embeddings(0, 1), ref.tensair_read_embeddings(0, 1)) <= TOL
    # after a batch from host memory (which the library prepares ahead of its turn, in buffers of its own) the entry
    # point still works in its array and the taps follow the last call
    for ctx in (ref, new):
        ctx.tensair_train_batch_host(0, np.ascontiguousarray(stream[1]), 3)
    toks = torch.from_numpy(stream[0]).cuda()
    torch.cuda.synchronize()
    l_ref, _ = ref.tensair_train_batch(0, toks, 4, want_loss=True)
    l_new, _ = new.tensair_train_batch_static(0, toks, 4, want_loss=True)
    assert l_new == pytest.approx(l_ref, rel=1e-12)
    assert np.array_equal(new.tensair_read_negatives(), ref.tensair_read_negatives())
    for which in (0, 1):
        assert rel_err(new.tensair_read_embeddings(0, which), ref.tensair_read_embeddings(0, which)) <= TOL


def test_static_scratch_entry_point_rejects_what_does_not_fit():
    import torch

    from paper_2211_10280_b200 import binding as B

    assert torch.cuda.is_available(), "this test needs a CUDA device"
    wl = synth.scaled(synth.MID, V=30_000, d=64, batch=16_384, k=15, batches=1)
    ctx = B.Context(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch, reduction=wl.reduction)
    before = ctx.tensair_read_embeddings(0, 0)
    toks = torch.from_numpy(synth.token_stream(wl, 0)[0]).cuda()
    with pytest.raises(B.TensairError) as ei:
        ctx.tensair_train_batch_static(0, toks, 0)
    assert ei.value.code == B.ENOMEM and "built-in array holds" in str(ei.value)
    assert np.array_equal(ctx.tensair_read_embeddings(0, 0), before)
    ctx.tensair_train_batch(0, toks, 0, want_loss=True)      # the ordinary entry point still serves it
