"""The oracle fanned out over processes gives what the sequential oracle gives, bit for bit."""
import numpy as np

import oracle
from oracle import fanout


def test_fanout_equals_sequential():
    rng = np.random.default_rng(4)
    B, N, V = 11, 3, 300
    lp = rng.normal(0, 2, (B, N, V)).astype(np.float32)
    lq = (lp + rng.normal(0, 1, (B, N, V))).astype(np.float32)
    un = rng.random((B, N, 5)).astype(np.float32)
    T = np.linspace(0.5, 1.5, B).astype(np.float32)
    kind = np.array([0, 0, 1], np.uint8)
    with fanout.Pool(3) as pool:
        assert pool.n == 3 and fanout.cores() >= 1
        for m in ("spechub", "rrs", "rrsw"):
            d_seq = oracle.draft_batch(m, lq, T, un)
            d_par = pool.draft_batch(m, lq, T, un)
            for k in d_seq:
                np.testing.assert_array_equal(d_seq[k], d_par[k], err_msg="%s %s" % (m, k))
            v_seq = oracle.verify_batch(m, lp, lq, T, d_seq["tokens"], un, kind)
            v_par = pool.verify_batch(m, lp, lq, T, d_seq["tokens"], un, kind)
            assert v_seq.tobytes() == v_par.tobytes()


def test_fanout_without_shared_memory(monkeypatch):
    """Hosts whose /dev/shm is missing or small: the rows travel with the jobs, same results."""
    rng = np.random.default_rng(6)
    lq = rng.normal(0, 2, (5, 2, 64)).astype(np.float32)
    un = rng.random((5, 2, 5)).astype(np.float32)
    with fanout.Pool(2) as pool:
        def no_shm(arrays):
            raise OSError("no shared memory here")
        monkeypatch.setattr(pool, "_share", no_shm)
        d = pool.draft_batch("spechub", lq, 1.0, un)
    ref = oracle.draft_batch("spechub", lq, 1.0, un)
    for k in ref:
        np.testing.assert_array_equal(ref[k], d[k])
