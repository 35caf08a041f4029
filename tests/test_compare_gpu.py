"""The three-method calls (mdsd_compare_*) against the CPU oracle, and bit for bit against the
per-method calls they stand for."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

import oracle  # noqa: E402
import workloads  # noqa: E402
import parity  # noqa: E402

METHODS = ("spechub", "rrs", "rrsw")
NODE_KEYS = ("accept_idx", "token", "hub", "beta", "rate", "status")
SEQ_KEYS = ("n_accepted", "n_emitted", "path_nodes", "path_tokens")


@pytest.fixture(scope="module")
def sh():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2411_05289_b200 as lib

    lib.load_library()
    return lib


def bits(t):
    t = t.detach().cpu().numpy()
    return t.view(np.int32) if t.dtype == np.float32 else t


def separate_draft(sh, m, tq, und, tree, T):
    if m == "spechub":
        return sh.spechub_draft_sample(tq, und, tree, T)
    return sh.rrs_draft_sample(tq, und, tree, m == "rrsw", T)


def separate_verify(sh, m, tp, tq, tok, und, tree, T, probabilities=True):
    if m == "spechub":
        return sh.spechub_verify_tree(tp, tq, tok, und, tree, T, probabilities=probabilities)
    return sh.rrs_verify_tree(tp, tq, tok, und, tree, m == "rrsw", T, probabilities=probabilities)


def make_case(V, dtype, seed, B=5, N=7):
    rng = np.random.default_rng(seed)
    lp = rng.normal(0, 2.0, (B, N, V)).astype(np.float32)
    lq = lp + rng.normal(0, 1.0, (B, N, V)).astype(np.float32)
    lq[0, 1] = lp[0, 1]                                    # p = q
    lq[1, 2] = -np.inf; lq[1, 2, V - 1] = 0.0              # one-hot q
    lq[2, 0] = -60.0; lq[2, 0, V // 2] = 0.0               # nearly one-hot q
    lp[3, 3, : V // 2] = -np.inf; lq[3, 3, V // 2:] = -np.inf   # disjoint supports
    lp[4, 4] = np.round(lp[4, 4] * 2) / 2; lq[4, 4] = np.round(lq[4, 4] * 2) / 2   # many ties
    lq[4, 5, 7] = lq[4, 5].max() + 9.0                     # peaked draft
    lp[2, 6, 3] = np.nan                                   # flagged target row
    lq[3, 6, 9] = np.inf                                   # flagged draft row
    lp, lq = workloads.round_to_storage(lp, dtype), workloads.round_to_storage(lq, dtype)
    un = rng.integers(0, 1 << 24, (B, N, 5)).astype(np.float32) * np.float32(2.0 ** -24)
    return lp, lq, un


@pytest.mark.parametrize("paper", [False, True])
@pytest.mark.parametrize("V,dtype", [(1000, "fp32"), (4096, "bf16"), (8192, "bf16"), (12344, "bf16"),
                                     (40000, "bf16"), (81920, "bf16")])
def test_compare_calls(sh, V, dtype, paper):
    lp, lq, un = make_case(V, dtype, V + 29)
    B, N, _ = lp.shape
    T = np.array([1.0, 0.6, 1.3, 0.8, 1.0], np.float32)
    Tt = torch.from_numpy(T).cuda()
    tp, tq, und = workloads.to_device(lp, dtype), workloads.to_device(lq, dtype), torch.from_numpy(un).cuda()
    tree = sh.Tree.heap(N, leaves_sample=paper)
    kind = workloads.paper_node_kind(N) if paper else None

    # draft step: against the per-method calls bit for bit, and against the oracle
    dall = sh.mdsd_compare_draft_sample(tq, und, tree, Tt)
    torch.cuda.synchronize()
    oracle_tokens = {}
    for m in METHODS:
        dsep = separate_draft(sh, m, tq, und, tree, Tt)
        for k in dsep:
            np.testing.assert_array_equal(bits(dall[m][k]), bits(dsep[k]), err_msg="draft %s %s" % (m, k))
        _, od = parity.check_draft(m, lq, T, un, parity.to_numpy(dall[m]), label="compare-draft")
        oracle_tokens[m] = od["tokens"].copy()

    # verification on the oracle's drafts
    toks = {m: torch.from_numpy(oracle_tokens[m]).cuda() for m in METHODS}
    vall = sh.mdsd_compare_verify_tree(tp, tq, toks, und, tree, Tt)
    torch.cuda.synchronize()
    for m in METHODS:
        vsep = separate_verify(sh, m, tp, tq, toks[m], und, tree, Tt)
        for k in NODE_KEYS + SEQ_KEYS:
            np.testing.assert_array_equal(bits(vall[m][k]), bits(vsep[k]), err_msg="verify %s %s" % (m, k))
        out = parity.to_numpy(vall[m])
        parity.check_verify(m, lp, lq, T, oracle_tokens[m], un, kind, out, label="compare-verify")
        w = oracle.walk(out["accept_idx"], out["token"], tree.levels, node_kind=kind)
        for k in SEQ_KEYS:
            np.testing.assert_array_equal(out[k], w[k], err_msg="walk %s %s" % (m, k))

    # the same step with the draft statistics handed from the draft call to verification: one record per
    # row serves the three methods; the per-method *_stats calls bit for bit, and the oracle
    dall2 = sh.mdsd_compare_draft_sample_stats(tq, und, tree, Tt)
    stats = dall2.pop("stats")
    for m in METHODS:
        for k in dall[m]:
            np.testing.assert_array_equal(bits(dall2[m][k]), bits(dall[m][k]), err_msg="draft+stats %s %s" % (m, k))
        if m == "spechub":
            dsep = sh.spechub_draft_sample_stats(tq, und, tree, Tt)
        else:
            dsep = sh.rrs_draft_sample_stats(tq, und, tree, m == "rrsw", Tt)
        np.testing.assert_array_equal(bits(dsep["stats"]), bits(stats), err_msg="records %s" % m)
    vall2 = sh.mdsd_compare_verify_tree_stats(tp, tq, stats, toks, und, tree, Tt)
    torch.cuda.synchronize()
    for m in METHODS:
        if m == "spechub":
            vsep = sh.spechub_verify_tree_stats(tp, tq, stats, toks[m], und, tree, Tt)
        else:
            vsep = sh.rrs_verify_tree_stats(tp, tq, stats, toks[m], und, tree, m == "rrsw", Tt)
        for k in NODE_KEYS + SEQ_KEYS:
            np.testing.assert_array_equal(bits(vall2[m][k]), bits(vsep[k]), err_msg="verify+stats %s %s" % (m, k))
        parity.check_verify(m, lp, lq, T, oracle_tokens[m], un, kind, parity.to_numpy(vall2[m]),
                            label="compare-verify+stats")

    # without probability buffers: same decisions, tokens and walks
    lite = sh.mdsd_compare_verify_tree(tp, tq, toks, und, tree, Tt, probabilities=False)
    for m in METHODS:
        for k in ("accept_idx", "token", "hub", "status") + SEQ_KEYS:
            np.testing.assert_array_equal(bits(lite[m][k]), bits(vall[m][k]), err_msg="lite %s %s" % (m, k))


def test_compare_calls_reject_more_than_two_drafts(sh):
    tq = torch.zeros((1, 4, 8192), dtype=torch.bfloat16, device="cuda")
    tree = sh.Tree.kary(3, 2)
    with pytest.raises(ValueError):
        sh.mdsd_compare_draft_sample(tq, torch.zeros((1, 4, 7), device="cuda"), tree, 1.0)


def test_compare_calls_on_an_empty_batch(sh):
    tq = torch.empty((0, 7, 8192), dtype=torch.bfloat16, device="cuda")
    un = torch.empty((0, 7, 5), dtype=torch.float32, device="cuda")
    tree = sh.Tree.heap(7)
    d = sh.mdsd_compare_draft_sample(tq, un, tree, 1.0)
    out = sh.mdsd_compare_verify_tree(tq, tq, {m: d[m]["tokens"] for m in METHODS}, un, tree, 1.0)
    assert out["spechub"]["token"].shape == (0, 7)
