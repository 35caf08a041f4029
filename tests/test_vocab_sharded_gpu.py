"""Vocabulary-sharded SpecHub: the ranks' phases run in lockstep on one GPU (the exchanges become a
stack and an element-wise maximum), and the result is compared with the CPU oracle on the whole
rows.  No kernel waits on another: each phase is an ordinary launch."""
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


def make_case(V, dtype, seed, B=4, N=7):
    rng = np.random.default_rng(seed)
    lp = rng.normal(0, 2.0, (B, N, V)).astype(np.float32)
    lq = lp + rng.normal(0, 1.0, (B, N, V)).astype(np.float32)
    lq[0, 1] = lp[0, 1]                                    # p = q
    lq[1, 2] = -np.inf; lq[1, 2, V - 1] = 0.0              # one-hot q on the last rank
    lq[2, 0] = -60.0; lq[2, 0, V // 2] = 0.0               # nearly one-hot q
    lp[3, 3, : V // 2] = -np.inf; lq[3, 3, V // 2:] = -np.inf   # disjoint supports: whole slices empty
    lp[1, 4] = np.round(lp[1, 4] * 2) / 2; lq[1, 4] = np.round(lq[1, 4] * 2) / 2   # ties across ranks
    lq[0, 5, 7] = lq[0, 5].max() + 9.0                     # peaked draft
    lp[2, 6, 3] = np.nan                                   # flagged target row
    lq[3, 6, V - 2] = np.inf                               # flagged draft row
    lp, lq = workloads.round_to_storage(lp, dtype), workloads.round_to_storage(lq, dtype)
    un = rng.integers(0, 1 << 24, (B, N, 5)).astype(np.float32) * np.float32(2.0 ** -24)
    return lp, lq, un


def lockstep_draft(vs, slices_q, und, tree, shards, T):
    ranks = [vs.ShardedDraft(q, und, tree, s, T) for q, (s, _) in zip(slices_q, shards)]
    g = torch.stack([r.stats() for r in ranks])
    cand = torch.stack([r.candidates(g) for r in ranks]).max(0).values
    return [r.finish(cand) for r in ranks]


def lockstep_verify(vs, slices_p, slices_q, tok, und, tree, shards, T):
    ranks = [vs.ShardedVerify(p, q, tok, und, tree, s, T) for p, q, (s, _) in zip(slices_p, slices_q, shards)]
    g = torch.stack([r.stats() for r in ranks])
    gs = torch.stack([r.sums(g) for r in ranks])
    tokmax = torch.stack([r.decide(gs) for r in ranks]).max(0).values
    return [r.walk(tokmax.clone()) for r in ranks]


@pytest.mark.parametrize("paper", [False, True])
@pytest.mark.parametrize("nranks", [1, 2, 3, 8])
@pytest.mark.parametrize("V,dtype", [(1000, "fp32"), (9001, "bf16"), (40000, "bf16")])
def test_sharded_matches_oracle(sh, V, dtype, nranks, paper):
    from paper_2411_05289_b200 import vocab_sharded as vs

    lp, lq, un = make_case(V, dtype, V + nranks)
    B, N, _ = lp.shape
    T = np.array([1.0, 0.6, 1.3, 0.8], np.float32)
    Tt = torch.from_numpy(T).cuda()
    tp, tq, und = workloads.to_device(lp, dtype), workloads.to_device(lq, dtype), torch.from_numpy(un).cuda()
    tree = sh.Tree.heap(N, leaves_sample=paper)
    kind = workloads.paper_node_kind(N) if paper else None
    shards = vs.even_shards(V, nranks)
    # views into the full rows: slice starts are unaligned whenever an offset is odd
    sp = [tp[:, :, s.id_offset:s.id_offset + w] for s, w in shards]
    sq = [tq[:, :, s.id_offset:s.id_offset + w] for s, w in shards]

    drafts = lockstep_draft(vs, sq, und, tree, shards, Tt)
    for d in drafts[1:]:
        for k in d:
            assert torch.equal(d[k], drafts[0][k]), "ranks disagree on draft %s" % k
    d0 = parity.to_numpy(drafts[0])
    d0["prob"] = None
    _, od = parity.check_draft("spechub", lq, T, un, d0, label="sharded-draft-%d" % nranks)

    tok = torch.from_numpy(od["tokens"].copy()).cuda()
    outs = lockstep_verify(vs, sp, sq, tok, und, tree, shards, Tt)
    torch.cuda.synchronize()
    for o in outs[1:]:
        for k in o:
            a, b = o[k], outs[0][k]
            assert torch.equal(a.view(torch.int32) if a.dtype == torch.float32 else a,
                               b.view(torch.int32) if b.dtype == torch.float32 else b), "ranks disagree on %s" % k
    out = parity.to_numpy(outs[0])
    assert (out["token"] >= -1).all(), "a drawn token was not delivered by its owner"
    parity.check_verify("spechub", lp, lq, T, od["tokens"], un, kind, out, label="sharded-verify-%d" % nranks)
    w = oracle.walk(out["accept_idx"], out["token"], tree.levels, node_kind=kind)
    for k in ("n_accepted", "n_emitted", "path_nodes", "path_tokens"):
        np.testing.assert_array_equal(out[k], w[k], err_msg="walk %s" % k)


def lockstep_rrs_draft(vs, slices_q, und, tree, shards, T, wo):
    ranks = [vs.ShardedRrsDraft(q, und, tree, s, wo, T) for q, (s, _) in zip(slices_q, shards)]
    g = torch.stack([r.stats() for r in ranks])
    res = [r.candidates(g) for r in ranks]
    cand = torch.stack([c for c, _ in res]).max(0).values
    ex1 = torch.stack([e for _, e in res]).max(0).values
    if wo:
        cand = torch.stack([r.second(cand, ex1) for r in ranks]).max(0).values
    return [r.finish(cand) for r in ranks]


def lockstep_rrs_verify(vs, slices_p, slices_q, tok, und, tree, shards, T, wo):
    ranks = [vs.ShardedRrsVerify(p, q, tok, und, tree, s, wo, T) for p, q, (s, _) in zip(slices_p, slices_q, shards)]
    g = torch.stack([r.stats() for r in ranks])
    gs = torch.stack([r.sums(g) for r in ranks])
    gw = torch.stack([r.w2(gs) for r in ranks])
    tokmax = torch.stack([r.decide(gw) for r in ranks]).max(0).values
    return [r.walk(tokmax.clone()) for r in ranks]


@pytest.mark.parametrize("wo", [False, True])
@pytest.mark.parametrize("paper", [False, True])
@pytest.mark.parametrize("nranks", [1, 3, 8])
@pytest.mark.parametrize("V,dtype", [(1000, "fp32"), (9001, "bf16"), (40000, "bf16")])
def test_sharded_rrs_matches_oracle(sh, V, dtype, nranks, paper, wo):
    from paper_2411_05289_b200 import vocab_sharded as vs

    method = "rrsw" if wo else "rrs"
    lp, lq, un = make_case(V, dtype, V + nranks + 100)
    B, N, _ = lp.shape
    T = np.array([1.0, 0.6, 1.3, 0.8], np.float32)
    Tt = torch.from_numpy(T).cuda()
    tp, tq, und = workloads.to_device(lp, dtype), workloads.to_device(lq, dtype), torch.from_numpy(un).cuda()
    tree = sh.Tree.heap(N, leaves_sample=paper)
    kind = workloads.paper_node_kind(N) if paper else None
    shards = vs.even_shards(V, nranks)
    sp = [tp[:, :, s.id_offset:s.id_offset + w] for s, w in shards]
    sq = [tq[:, :, s.id_offset:s.id_offset + w] for s, w in shards]

    drafts = lockstep_rrs_draft(vs, sq, und, tree, shards, Tt, wo)
    for d in drafts[1:]:
        for k in d:
            assert torch.equal(d[k], drafts[0][k]), "ranks disagree on draft %s" % k
    d0 = parity.to_numpy(drafts[0])
    _, od = parity.check_draft(method, lq, T, un, d0, label="sharded-%s-draft-%d" % (method, nranks))

    tok = torch.from_numpy(od["tokens"].copy()).cuda()
    outs = lockstep_rrs_verify(vs, sp, sq, tok, und, tree, shards, Tt, wo)
    torch.cuda.synchronize()
    for o in outs[1:]:
        for k in o:
            a, b = o[k], outs[0][k]
            assert torch.equal(a.view(torch.int32) if a.dtype == torch.float32 else a,
                               b.view(torch.int32) if b.dtype == torch.float32 else b), "ranks disagree on %s" % k
    out = parity.to_numpy(outs[0])
    assert (out["token"] >= -1).all(), "a drawn token was not delivered by its owner"
    parity.check_verify(method, lp, lq, T, od["tokens"], un, kind, out, label="sharded-%s-verify-%d" % (method, nranks))
    w = oracle.walk(out["accept_idx"], out["token"], tree.levels, node_kind=kind)
    for k in ("n_accepted", "n_emitted", "path_nodes", "path_tokens"):
        np.testing.assert_array_equal(out[k], w[k], err_msg="walk %s" % k)


def test_one_rank_equals_the_unsharded_calls(sh):
    """With a single rank the phases see the whole row: decisions and tokens equal the one-call path."""
    from paper_2411_05289_b200 import vocab_sharded as vs

    lp, lq, un = make_case(5000, "fp32", 77)
    tp, tq, und = workloads.to_device(lp, "fp32"), workloads.to_device(lq, "fp32"), torch.from_numpy(un).cuda()
    tree = sh.Tree.heap(7)
    shards = vs.even_shards(5000, 1)
    d = lockstep_draft(vs, [tq], und, tree, shards, 1.0)[0]
    ref = sh.spechub_draft_sample(tq, und, tree, 1.0)
    for k in ("tokens", "hub", "status"):
        assert torch.equal(d[k], ref[k]), k
    o = lockstep_verify(vs, [tp], [tq], ref["tokens"], und, tree, shards, 1.0)[0]
    full = sh.spechub_verify_tree(tp, tq, ref["tokens"], und, tree, 1.0)
    for k in ("accept_idx", "token", "hub", "status", "n_accepted", "n_emitted", "path_nodes", "path_tokens"):
        assert torch.equal(o[k], full[k]), k
    for k in ("beta", "rate"):
        torch.testing.assert_close(o[k], full[k], rtol=1e-5, atol=1e-6)


def test_shard_argument_errors(sh):
    from paper_2411_05289_b200 import vocab_sharded as vs

    tq = torch.zeros((1, 3, 64), device="cuda")
    un = torch.zeros((1, 3, 5), device="cuda")
    tree = sh.Tree.heap(3)
    for bad in (vs.Shard(2, 2, 0, 128), vs.Shard(0, 65, 0, 128), vs.Shard(0, 2, 100, 128), vs.Shard(0, 1, -1, 64)):
        with pytest.raises(sh.SpecHubError):
            vs.ShardedDraft(tq, un, tree, bad, 1.0).stats()


def test_sharded_drivers_on_a_stream_that_is_not_current(sh):
    """The torch.distributed drivers mix launches, allocations and collectives; a caller's stream must
    carry all of them.  One rank (NCCL, world size 1) holding the whole vocabulary: the results on a
    side stream equal those on the current stream, and those of the plain calls."""
    import os
    import socket

    import torch.distributed as dist

    from paper_2411_05289_b200 import vocab_sharded as vs

    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        lp, lq, un = make_case(9001, "bf16", 5)
        tp, tq = workloads.to_device(lp, "bf16"), workloads.to_device(lq, "bf16")
        und = torch.from_numpy(un).cuda()
        tree = sh.Tree.heap(7)
        shard, _ = vs.even_shards(9001, 1)[0]
        T = torch.tensor([1.0, 0.7, 1.3, 0.9], device="cuda")
        ref_d = vs.spechub_draft_sample_sharded(tq, und, tree, shard, T)
        ref_v = vs.spechub_verify_tree_sharded(tp, tq, ref_d["tokens"], und, tree, shard, T)
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        for rep in range(3):
            d = vs.spechub_draft_sample_sharded(tq, und, tree, shard, T, stream=side)
            v = vs.spechub_verify_tree_sharded(tp, tq, d["tokens"], und, tree, shard, T, stream=side)
        side.synchronize()
        assert torch.equal(d["tokens"], ref_d["tokens"])
        for k in ("accept_idx", "token", "n_accepted", "n_emitted", "path_tokens"):
            assert torch.equal(v[k], ref_v[k]), k
        # the plain calls with an explicit stream and a per-sequence temperature tensor (a temporary of the call)
        for rep in range(3):
            pd = sh.spechub_draft_sample(tq, und, tree, T.double(), stream=side)
            pv = sh.spechub_verify_tree(tp, tq, pd["tokens"], und, tree, T.double(), stream=side)
        side.synchronize()
        cur = sh.spechub_verify_tree(tp, tq, sh.spechub_draft_sample(tq, und, tree, T)["tokens"], und, tree, T)
        torch.cuda.synchronize()
        for k in ("accept_idx", "token", "n_emitted"):
            assert torch.equal(pv[k], cur[k]), k
    finally:
        dist.destroy_process_group()
