"""Helpers shared by the GPU parity tests: paired oracle / CUDA runs and the error measure."""
import numpy as np

from oracle import Oracle
from paper_2211_10280_b200 import synth


def rel_err(got: np.ndarray, want: np.ndarray) -> float:
    """max_i |got_i - want_i| / max(|want_i|, tau), tau = 1e-2 * rms(want).

    Output rows start at zero, so a plain relative error is undefined on them; the floor tau ties the
    measure to the typical magnitude of the array under comparison.
    """
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    if want.size == 0:
        return 0.0
    tau = 1e-2 * float(np.sqrt(np.mean(want * want)))
    if tau == 0.0:
        return 0.0 if np.array_equal(got, want) else float("inf")
    return float(np.max(np.abs(got - want) / np.maximum(np.abs(want), tau)))


def make_pair(wl: synth.Workload, counts=None, init_in=None, init_out=None, batch=None, max_grad_buffer=1):
    """An oracle and a CUDA context with identical configuration and initial state."""
    from paper_2211_10280_b200 import binding as B

    kw = dict(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=batch or wl.batch, W=wl.W, lr=wl.lr,
              max_delay=wl.max_delay, seed=wl.seed, counts=counts, init_in=init_in, init_out=init_out,
              reduction=wl.reduction, max_grad_buffer=max_grad_buffer)
    return Oracle(**kw), B.Context(**kw)


def tables(obj, replica, gpu: bool):
    if gpu:
        return obj.tensair_read_embeddings(replica, 0), obj.tensair_read_embeddings(replica, 1)
    return obj.read_embeddings(replica, 0), obj.read_embeddings(replica, 1)


def compare_tables(o, g, replica, tol):
    oi, oo = tables(o, replica, False)
    gi, go = tables(g, replica, True)
    e_in, e_out = rel_err(gi, oi), rel_err(go, oo)
    assert e_in <= tol and e_out <= tol, (e_in, e_out, tol)
    return e_in, e_out


def compare_message(o, g, replica, step, tol):
    om = o.read_message(replica, step)
    gm = g.tensair_read_message(replica, step)
    assert om is not None and gm is not None
    assert np.array_equal(om[0], gm[0]), "message row ids differ"
    e = rel_err(gm[1], om[1])
    assert e <= tol, (e, tol)
    return e
