"""spechub_verify_tree_static: the verification entry point for callers that cannot allocate
device memory (a serving process whose pools own the whole GPU, code inside another framework's
memory plan, a loop that may not enter the driver's allocator).  It keeps its intermediate per-row
records in a static array inside the library, which every call on the device shares.

Checked here, through the C ABI: two calls in a row -- the second on other data and fewer rows, so
that anything left in the array by the first would show -- give what spechub_verify_tree gives
(decisions, tokens, hub, status and the walk equal; probabilities within the parity tolerance);
the results also pass the oracle comparison on a large-vocabulary bf16 shape; and a call beyond
the array's capacity is refused.  The file name sorts last on purpose: a run that stops at the
first failure has then already run every other test.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

import oracle  # noqa: E402
import workloads  # noqa: E402
import parity  # noqa: E402

INT_KEYS = ("accept_idx", "token", "hub", "status", "n_accepted", "n_emitted", "path_nodes", "path_tokens")


@pytest.fixture(scope="module")
def sh():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2411_05289_b200 as lib

    lib.load_library()
    return lib


def case(seed, B, N, V, dtype):
    rng = np.random.default_rng(seed)
    lp = rng.normal(0, 2.0, (B, N, V)).astype(np.float32)
    lq = lp + rng.normal(0, 1.0, (B, N, V)).astype(np.float32)
    lq[0, 1] = lp[0, 1]                           # p = q
    lq[B - 1, 2] = -np.inf; lq[B - 1, 2, 5] = 0.0  # one-hot q
    lp[0, 0, 3] = np.nan                          # flagged row
    lp, lq = workloads.round_to_storage(lp, dtype), workloads.round_to_storage(lq, dtype)
    un = rng.integers(0, 1 << 24, (B, N, 5)).astype(np.float32) * np.float32(2.0 ** -24)
    return lp, lq, un


def run_both(sh, lp, lq, un, dtype, paper):
    B, N, V = lp.shape
    tp, tq, und = workloads.to_device(lp, dtype), workloads.to_device(lq, dtype), torch.from_numpy(un).cuda()
    tree = sh.Tree.heap(N, leaves_sample=paper)
    tok = sh.spechub_draft_sample(tq, und, tree, 1.0)["tokens"]
    ref = sh.spechub_verify_tree(tp, tq, tok, und, tree, 1.0)
    got = sh.spechub_verify_tree_static(tp, tq, tok, und, tree, 1.0)
    torch.cuda.synchronize()
    return parity.to_numpy(ref), parity.to_numpy(got), parity.to_numpy({"tokens": tok})["tokens"]


def test_two_calls_in_a_row_match_the_allocating_entry_point(sh):
    # shapes that the existing entry point runs through the same per-row arithmetic
    for seed, B, N, V, dtype, paper in ((1, 6, 7, 5000, "fp32", False), (2, 3, 3, 4096, "bf16", True)):
        lp, lq, un = case(seed, B, N, V, dtype)
        ref, got, _ = run_both(sh, lp, lq, un, dtype, paper)
        for k in INT_KEYS:
            np.testing.assert_array_equal(got[k], ref[k], err_msg="%s (call with seed %d)" % (k, seed))
        for k in ("beta", "rate"):
            np.testing.assert_allclose(got[k], ref[k], rtol=parity.RTOL, atol=parity.ATOL, err_msg=k)
        assert (ref["accept_idx"] >= 0).any() and (ref["accept_idx"] < 0).any()


def test_large_vocabulary_rows_pass_the_oracle_comparison(sh):
    # here the existing entry point sums in another order, so both are held against the oracle
    lp, lq, un = case(3, 4, 7, 40000, "bf16")
    for paper in (False, True):
        ref, got, tok = run_both(sh, lp, lq, un, "bf16", paper)
        kind = workloads.paper_node_kind(7) if paper else None
        parity.check_verify("spechub", lp, lq, 1.0, tok, un, kind, got, label="static")
        w = oracle.walk(got["accept_idx"], got["token"], 3, node_kind=kind)
        for k in ("n_accepted", "n_emitted", "path_nodes", "path_tokens"):
            np.testing.assert_array_equal(got[k], w[k], err_msg=k)
        np.testing.assert_allclose(got["rate"], ref["rate"], rtol=parity.RTOL, atol=parity.ATOL)


def test_more_rows_than_the_static_array_holds_are_refused(sh):
    from paper_2411_05289_b200.binding import STATIC_MAX_ROWS

    B, N, V = STATIC_MAX_ROWS // 3 + 1, 3, 64
    z = torch.zeros((B, N, V), device="cuda")
    un = torch.zeros((B, N, 5), device="cuda")
    tok = torch.zeros((B, N, 2), dtype=torch.int32, device="cuda")
    with pytest.raises(sh.SpecHubError) as e:
        sh.spechub_verify_tree_static(z, z, tok, un, sh.Tree.heap(3), 1.0)
    assert e.value.code == -10 and "SPECHUB_STATIC_MAX_ROWS" in str(e.value)
