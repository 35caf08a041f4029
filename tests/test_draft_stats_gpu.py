"""Draft statistics handed from the draft step to verification (spechub_draft_sample_stats ->
spechub_verify_tree_stats and the RRS pair): the records are refused when they are not the row's, ignored
where no kernel uses them, and on the large-vocabulary bf16 shapes verification with them agrees with the
plain call.  Parity with the oracle of this path is part of every case of test_parity_gpu.py."""
import numpy as np
import pytest
import torch

import workloads

pytestmark = pytest.mark.gpu

ST_STATS = 64


@pytest.fixture(scope="module")
def sh():
    import paper_2411_05289_b200 as lib

    lib.load_library()
    return lib


def problem(V, dtype, seed, B=4, N=7):
    rng = np.random.default_rng(seed)
    lp = rng.normal(0, 2.0, (B, N, V)).astype(np.float32)
    lq = lp + rng.normal(0, 1.0, (B, N, V)).astype(np.float32)
    un = (rng.integers(0, 1 << 24, (B, N, 5)).astype(np.float32) * np.float32(2.0 ** -24))
    return workloads.to_device(lp, dtype, "cuda"), workloads.to_device(lq, dtype, "cuda"), torch.from_numpy(un).cuda()


def draft(sh, m, tq, un, tree, T=1.0, stats=True):
    if m == "spechub":
        return (sh.spechub_draft_sample_stats if stats else sh.spechub_draft_sample)(tq, un, tree, T)
    return (sh.rrs_draft_sample_stats if stats else sh.rrs_draft_sample)(tq, un, tree, m == "rrsw", T)


def verify(sh, m, tp, tq, d, un, tree, T=1.0, stats=None):
    if m == "spechub":
        if stats is None:
            return sh.spechub_verify_tree(tp, tq, d["tokens"], un, tree, T)
        return sh.spechub_verify_tree_stats(tp, tq, stats, d["tokens"], un, tree, T)
    if stats is None:
        return sh.rrs_verify_tree(tp, tq, d["tokens"], un, tree, m == "rrsw", T)
    return sh.rrs_verify_tree_stats(tp, tq, stats, d["tokens"], un, tree, m == "rrsw", T)


@pytest.mark.parametrize("m", ["spechub", "rrs", "rrsw"])
@pytest.mark.parametrize("V", [8192, 32000, 128256])
def test_verification_with_statistics_agrees_with_the_plain_call(sh, m, V):
    tp, tq, un = problem(V, "bf16", V + 1)
    tree = sh.Tree.heap(7)
    d = draft(sh, m, tq, un, tree)
    plain = verify(sh, m, tp, tq, d, un, tree)
    withs = verify(sh, m, tp, tq, d, un, tree, stats=d["stats"])
    torch.cuda.synchronize()
    assert int((withs["status"] & ST_STATS).sum()) == 0
    # the draft row's normaliser is summed in another order: probabilities agree to rounding, and a
    # decision can differ only on a row whose test sits on its threshold (none in this seeded case)
    for k in ("beta", "rate"):
        torch.testing.assert_close(withs[k], plain[k], rtol=2e-5, atol=2e-6)
    for k in ("accept_idx", "token", "hub", "n_accepted", "n_emitted", "path_tokens"):
        assert torch.equal(withs[k], plain[k]), k


@pytest.mark.parametrize("m", ["spechub", "rrs", "rrsw"])
def test_records_of_other_logits_or_another_temperature_are_refused(sh, m):
    V = 16384
    tp, tq, un = problem(V, "bf16", 5)
    _, tq_other, _ = problem(V, "bf16", 6)
    tree = sh.Tree.heap(7)
    d = draft(sh, m, tq, un, tree)
    d_other = draft(sh, m, tq_other, un, tree)
    # (a) records made from other draft logits: the recorded maximum is not what the row holds at the
    # recorded argmax (with 16384 random logits per row a chance match does not happen in this seed)
    out = verify(sh, m, tp, tq, d, un, tree, stats=d_other["stats"])
    torch.cuda.synchronize()
    assert bool(((out["status"] & ST_STATS) != 0).all())
    assert bool((out["token"] == -1).all()) and bool((out["accept_idx"] == -1).all())
    # (b) records made at another temperature
    d_t = draft(sh, m, tq, un, tree, T=0.7)
    out = verify(sh, m, tp, tq, d, un, tree, T=1.0, stats=d_t["stats"])
    torch.cuda.synchronize()
    assert bool(((out["status"] & ST_STATS) != 0).all())
    # (c) a cleared buffer
    out = verify(sh, m, tp, tq, d, un, tree, stats=torch.zeros_like(d["stats"]))
    torch.cuda.synchronize()
    assert bool(((out["status"] & ST_STATS) != 0).all())


@pytest.mark.parametrize("V,dtype", [(1000, "fp32"), (4096, "bf16"), (9001, "bf16")])
def test_shapes_without_a_statistics_kernel_clear_and_ignore_the_records(sh, V, dtype):
    tp, tq, un = problem(V, dtype, V)
    tree = sh.Tree.heap(7)
    for m in ("spechub", "rrs", "rrsw"):
        d = draft(sh, m, tq, un, tree)
        assert int(d["stats"].abs().sum()) == 0
        plain = verify(sh, m, tp, tq, d, un, tree)
        withs = verify(sh, m, tp, tq, d, un, tree, stats=d["stats"])
        torch.cuda.synchronize()
        for k in plain:
            assert torch.equal(plain[k], withs[k]), (m, k)


def test_a_forced_split_neither_writes_nor_reads_records(sh):
    tp, tq, un = problem(16384, "bf16", 9)
    tree = sh.Tree.heap(7)
    sh.set_row_split(2)
    try:
        d = draft(sh, "spechub", tq, un, tree)
        assert int(d["stats"].abs().sum()) == 0
        plain = verify(sh, "spechub", tp, tq, d, un, tree)
        withs = verify(sh, "spechub", tp, tq, d, un, tree, stats=d["stats"])
        torch.cuda.synchronize()
        for k in plain:
            assert torch.equal(plain[k], withs[k]), k
    finally:
        sh.set_row_split(0)


def test_nonfinite_draft_rows_keep_their_status(sh):
    V = 16384
    tp, tq, un = problem(V, "bf16", 11)
    tq[0, 1, 5] = float("nan")
    tq[1, 2, :] = float("-inf")
    tq[2, 3, 7] = float("inf")
    tree = sh.Tree.heap(7)
    for m in ("spechub", "rrs", "rrsw"):
        d = draft(sh, m, tq, un, tree)
        plain = verify(sh, m, tp, tq, d, un, tree)
        withs = verify(sh, m, tp, tq, d, un, tree, stats=d["stats"])
        torch.cuda.synchronize()
        assert torch.equal(plain["status"], withs["status"]), m
        assert torch.equal(plain["token"], withs["token"]), m


def test_records_are_reusable_and_the_buffer_is_checked(sh):
    tp, tq, un = problem(16384, "bf16", 13)
    tree = sh.Tree.heap(7)
    d = draft(sh, "spechub", tq, un, tree)
    a = verify(sh, "spechub", tp, tq, d, un, tree, stats=d["stats"])
    b = verify(sh, "spechub", tp, tq, d, un, tree, stats=d["stats"])
    torch.cuda.synchronize()
    for k in a:
        assert torch.equal(a[k], b[k]), k
    with pytest.raises(ValueError):
        verify(sh, "spechub", tp, tq, d, un, tree, stats=d["stats"][:8])


def test_more_than_two_drafts_neither_write_nor_read_records(sh):
    """k = 3 (RRS / RRSw only): the draft kernels of that path keep no statistics and its verification
    kernels take none; the *_stats calls are the plain calls."""
    rng = np.random.default_rng(21)
    tree = sh.Tree.kary(3, 3)
    B, N, V = 3, tree.nodes_of_complete_tree(), 16384
    lp = rng.normal(0, 2.0, (B, N, V)).astype(np.float32)
    lq = lp + rng.normal(0, 1.0, (B, N, V)).astype(np.float32)
    tp, tq = workloads.to_device(lp, "bf16", "cuda"), workloads.to_device(lq, "bf16", "cuda")
    un = torch.from_numpy(rng.integers(0, 1 << 24, (B, N, 7)).astype(np.float32) * np.float32(2.0 ** -24)).cuda()
    for wo in (False, True):
        d = sh.rrs_draft_sample_stats(tq, un, tree, wo)
        plain_d = sh.rrs_draft_sample(tq, un, tree, wo)
        assert int(d["stats"].abs().sum()) == 0
        assert torch.equal(d["tokens"], plain_d["tokens"])
        a = sh.rrs_verify_tree(tp, tq, d["tokens"], un, tree, wo)
        b = sh.rrs_verify_tree_stats(tp, tq, d["stats"], d["tokens"], un, tree, wo)
        torch.cuda.synchronize()
        for k in a:
            assert torch.equal(a[k], b[k]), (wo, k)
