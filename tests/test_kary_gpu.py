"""Parity of RRS / RRSw with k > 2 drafts per node (Algorithm 1 for general k) against the oracle."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

import oracle  # noqa: E402
import workloads  # noqa: E402
import parity  # noqa: E402


@pytest.fixture(scope="module")
def sh():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2411_05289_b200 as lib

    lib.load_library()
    return lib


def close(g, o, cond, what, ctx):
    tol = parity.RTOL * np.abs(o) + parity.ATOL + parity.EPS * cond
    assert np.all(np.abs(g - o) <= tol), (what, ctx, g, o)


def check(sh, k, wo, lp, lq, dtype, T, un, levels, leaves):
    B, N, V = lp.shape
    tree = sh.Tree.kary(k, levels, leaves_sample=leaves)
    assert tree.nodes_of_complete_tree() == N
    kind = None
    if leaves:
        kind = np.zeros(N, np.uint8)
        kind[(k ** (levels - 1) - 1) // (k - 1):] = 1
    tp, tq = workloads.to_device(lp, dtype), workloads.to_device(lq, dtype)
    und = torch.from_numpy(un).cuda()
    d = parity.to_numpy(sh.rrs_draft_sample(tq, und, tree, wo, T))
    od = oracle.rrs_k_draft_batch(k, wo, lq, T, un)
    exact = near = 0
    for b in range(B):
        for n in range(N):
            if tuple(d["tokens"][b, n]) == tuple(od["tokens"][b, n]):
                exact += 1
                assert d["status"][b, n] == od["status"][b, n]
                continue
            # differing draws must each be admissible given the GPU's earlier draws
            q, _ = oracle.softmax(lq[b, n], T)
            w = q.copy()
            for i in range(k):
                x = int(d["tokens"][b, n, i])
                lo, hi = oracle.cdf_interval(w, x)
                assert lo - parity.NEAR <= un[b, n, i] <= hi + parity.NEAR, ("draft", b, n, i)
                if wo:
                    w[x] = 0.0
            near += 1
    tok = od["tokens"].copy()
    out = parity.to_numpy(sh.rrs_verify_tree(tp, tq, torch.from_numpy(tok).cuda(), und, tree, wo, T))
    torch.cuda.synchronize()
    ov = oracle.rrs_k_verify_batch(k, wo, lp, lq, T, tok, un, kind)
    for b in range(B):
        for n in range(N):
            ctx = "k=%d wo=%s b=%d n=%d V=%d" % (k, wo, b, n, V)
            if kind is not None and kind[n] == 1:
                if out["token"][b, n] != ov["token"][b, n]:
                    p, _ = oracle.softmax(lp[b, n], T)
                    lo, hi = oracle.cdf_interval(p, int(out["token"][b, n]))
                    assert lo - parity.NEAR <= un[b, n, 2 * k] <= hi + parity.NEAR, ctx
                continue
            close(out["beta"][b, n], ov["beta"][b, n], ov["cond"][b, n], "beta", ctx)
            close(out["rate"][b, n], ov["rate"][b, n], 0.0, "rate", ctx)
            same = out["accept_idx"][b, n] == ov["accept_idx"][b, n] and out["token"][b, n] == ov["token"][b, n]
            if same:
                exact += 1
                assert out["status"][b, n] | 16 == ov["status"][b, n] | 16, ctx
                continue
            # only allowed next to a threshold (band widened by the conditioning of that test)
            bands = [max(parity.NEAR, parity.EPS * c) for c in ov["cond"][b, n]] + [parity.NEAR]
            assert any(m <= bd for m, bd in zip(ov["margin"][b, n], bands)), (ctx, out["accept_idx"][b, n],
                                                                             ov["accept_idx"][b, n], ov["margin"][b, n])
            near += 1
    w = oracle.walk_k(k, out["accept_idx"], out["token"], levels, node_kind=kind)
    for key in ("n_accepted", "n_emitted", "path_nodes", "path_tokens"):
        np.testing.assert_array_equal(out[key], w[key], err_msg=key)
    return exact, near


@pytest.mark.parametrize("wo", [False, True])
@pytest.mark.parametrize("k,levels", [(3, 3), (4, 2), (8, 2)])
@pytest.mark.parametrize("V,dtype", [(5, "fp32"), (9, "fp32"), (1000, "fp32"), (4099, "bf16"), (8192, "bf16"),
                                     (32000, "bf16"), (40000, "bf16"), (131080, "bf16")])
def test_kary_parity(sh, k, levels, V, dtype, wo):
    if wo and V < k:
        pytest.skip("cannot draw k distinct tokens")
    if V > 32000 and (k, levels) != (3, 3):
        pytest.skip("the long rows (a row over 2 or 4 CTAs) are covered with the ternary tree")
    rng = np.random.default_rng(V * 31 + k * 7 + wo)
    N = (k ** levels - 1) // (k - 1)
    B = 3
    lp = rng.normal(0, 2.0, (B, N, V)).astype(np.float32)
    lq = lp + rng.normal(0, 0.8, (B, N, V)).astype(np.float32)
    lq[0, 0] = lp[0, 0]                              # p = q
    if V > 100:
        lq[1, 1] = -np.inf; lq[1, 1, 3] = 0.0        # one-hot q: without replacement runs dry
        lq[2, 0, :] = -50.0; lq[2, 0, :k - 1] = 0.0  # almost all mass on fewer tokens than drafts
    lp, lq = workloads.round_to_storage(lp, dtype), workloads.round_to_storage(lq, dtype)
    un = (rng.integers(0, 1 << 24, (B, N, 2 * k + 1)).astype(np.float32) * np.float32(2.0 ** -24))
    for leaves in (False, True):
        exact, near = check(sh, k, wo, lp, lq, dtype, 0.9, un, levels, leaves)
        assert exact > 0


def test_kary_argument_checks(sh):
    tree3 = sh.Tree.kary(3, 2)
    x = torch.zeros((1, 4, 64), device="cuda")
    with pytest.raises(ValueError):
        sh.spechub_draft_sample(x, torch.zeros((1, 4, 7), device="cuda"), tree3)
    with pytest.raises(ValueError):
        sh.rrs_draft_sample(x, torch.zeros((1, 4, 5), device="cuda"), tree3, False)
    import ctypes

    from paper_2411_05289_b200 import binding

    d, _ = binding._desc(x, tree3, 1.0)
    lib = sh.load_library()
    vp = ctypes.c_void_p
    un = torch.zeros((1, 4, 7), device="cuda")
    tk = torch.zeros((1, 4, 3), dtype=torch.int32, device="cuda")
    # SpecHub refuses k != 2 on the host
    assert lib.spechub_draft_sample(ctypes.byref(d), vp(x.data_ptr()), vp(un.data_ptr()), vp(tk.data_ptr()),
                                    None, None, None, None) == -3
    d.k = 9
    assert lib.rrs_draft_sample(ctypes.byref(d), vp(x.data_ptr()), vp(un.data_ptr()), 0, vp(tk.data_ptr()),
                                None, None) == -3
