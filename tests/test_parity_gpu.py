"""Parity of the CUDA library (through the C ABI) against the CPU oracle.

Small problems are compared row by row on every output; the five benchmark
configurations run on the GPU at full size, in the launch configuration the
benchmark times, and are compared on sampled rows.
"""
import os

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

import oracle  # noqa: E402
import workloads  # noqa: E402
import parity  # noqa: E402

METHODS = ("spechub", "rrs", "rrsw")


@pytest.fixture(scope="module")
def sh():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2411_05289_b200 as lib

    lib.load_library()
    return lib


@pytest.fixture(scope="module")
def pool():
    """The oracle on all host cores (started with spawn: CUDA is already up in this process)."""
    from oracle import fanout

    with fanout.Pool() as p:
        yield p


# Rows a full-size configuration may leave to the near-threshold rule.  Measured on configs 1-5: at
# most 0.43 % of the rows, all of them residual or draft draws whose uniform lies within 1e-6 of an
# edge of the oracle's CDF (tens of thousands of edges per row); no acceptance test was exempted.  A
# fraction far above that means the rule is hiding something.
MAX_EXEMPT_FRACTION = 0.02


def report(name, s):
    print("%s %r" % (name, s))
    assert s.wide_band == 0, "%s: %d rows needed the conditioning-widened band" % (name, s.wide_band)
    assert s.exempt_fraction() <= MAX_EXEMPT_FRACTION, (name, s.exempt_fraction())


def gpu_draft(sh, method, tq, un, tree, T):
    if method == "spechub":
        return sh.spechub_draft_sample(tq, un, tree, T)
    return sh.rrs_draft_sample(tq, un, tree, method == "rrsw", T)


def gpu_verify(sh, method, tp, tq, tok, un, tree, T, out=None):
    if method == "spechub":
        return sh.spechub_verify_tree(tp, tq, tok, un, tree, T, out=out)
    return sh.rrs_verify_tree(tp, tq, tok, un, tree, method == "rrsw", T, out=out)


def gpu_draft_stats(sh, method, tq, un, tree, T):
    if method == "spechub":
        return sh.spechub_draft_sample_stats(tq, un, tree, T)
    return sh.rrs_draft_sample_stats(tq, un, tree, method == "rrsw", T)


def gpu_verify_stats(sh, method, tp, tq, stats, tok, un, tree, T, out=None):
    if method == "spechub":
        return sh.spechub_verify_tree_stats(tp, tq, stats, tok, un, tree, T, out=out)
    return sh.rrs_verify_tree_stats(tp, tq, stats, tok, un, tree, method == "rrsw", T, out=out)


def padded(x, dtype, pad_to, device="cuda"):
    """Device copy of host fp32 [B][N][V] in the storage dtype; rows padded to a multiple of
    `pad_to` elements (0 = dense rows, which are unaligned when V is odd)."""
    B, N, V = x.shape
    t = workloads.to_device(x, dtype, device)
    if not pad_to:
        return t
    Vp = (V + pad_to - 1) // pad_to * pad_to
    buf = torch.full((B, N, Vp), float("nan"), dtype=t.dtype, device=device)
    buf[:, :, :V] = t
    return buf[:, :, :V]


def run_case(sh, lp, lq, dtype, T, un, paper_layout, pad_to=0, methods=METHODS, label=""):
    B, N, V = lp.shape
    Tt = torch.tensor(np.asarray(T, np.float32), device="cuda") if np.ndim(T) else float(T)
    tp, tq = padded(lp, dtype, pad_to), padded(lq, dtype, pad_to)
    und = torch.from_numpy(un).cuda()
    kind = workloads.paper_node_kind(N) if paper_layout else None
    tree = sh.Tree.heap(N, leaves_sample=paper_layout)
    total = parity.Stats()
    for m in methods:
        d = parity.to_numpy(gpu_draft(sh, m, tq, und, tree, Tt))
        st, od = parity.check_draft(m, lq, T, un, d, label=label)
        # verification parity is checked on the oracle's drafts so that both sides see the same pair
        tok = od["tokens"].copy()
        out = parity.to_numpy(gpu_verify(sh, m, tp, tq, torch.from_numpy(tok).cuda(), und, tree, Tt))
        torch.cuda.synchronize()
        sv, ov = parity.check_verify(m, lp, lq, T, tok, un, kind, out, label=label)
        w = oracle.walk(out["accept_idx"], out["token"], tree.levels, node_kind=kind)
        for k in ("n_accepted", "n_emitted", "path_nodes", "path_tokens"):
            np.testing.assert_array_equal(out[k], w[k], err_msg="%s walk %s" % (label, k))
        total.add(st).add(sv)
        if tree.k == 2:
            # the same step with the draft statistics handed from the draft call to verification: the draft
            # call's own outputs do not change, and verification meets the same bar against the same records
            ds = gpu_draft_stats(sh, m, tq, und, tree, Tt)
            stats_t = ds.pop("stats")
            ds = parity.to_numpy(ds)
            for k in d:
                np.testing.assert_array_equal(ds[k], d[k], err_msg="%s draft with statistics: %s" % (label, k))
            out2 = parity.to_numpy(gpu_verify_stats(sh, m, tp, tq, stats_t, torch.from_numpy(tok).cuda(), und, tree, Tt))
            torch.cuda.synchronize()
            sv2, _ = parity.check_verify(m, lp, lq, T, tok, un, kind, out2, label=label + "+stats", oracle_out=ov)
            w2 = oracle.walk(out2["accept_idx"], out2["token"], tree.levels, node_kind=kind)
            for k in ("n_accepted", "n_emitted", "path_nodes", "path_tokens"):
                np.testing.assert_array_equal(out2[k], w2[k], err_msg="%s+stats walk %s" % (label, k))
            total.add(sv2)
    return total


def random_logits(rng, B, N, V, dtype, sd=2.0, sigma=1.0):
    lp = rng.normal(0, sd, (B, N, V)).astype(np.float32)
    lq = lp + rng.normal(0, sigma, (B, N, V)).astype(np.float32)
    return workloads.round_to_storage(lp, dtype), workloads.round_to_storage(lq, dtype)


def random_uniforms(rng, B, N):
    return (rng.integers(0, 1 << 24, (B, N, 5)).astype(np.float32) * np.float32(2.0 ** -24))


# ------------------------------------------------------------------------------------------------
# small shapes: every tile boundary, ragged tails, unaligned rows, both dtypes, both layouts
# ------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("V", [2, 3, 5, 8, 33, 257, 1000, 1031, 4099, 9000, 20011])
def test_small_shapes(sh, V, dtype):
    rng = np.random.default_rng(V * 7 + (dtype == "bf16"))
    B, N = (3, 7) if V > 1000 else (6, 7)
    lp, lq = random_logits(rng, B, N, V, dtype)
    un = random_uniforms(rng, B, N)
    T = np.array([1.0, 0.6, 1.3, 0.8, 1.0, 2.0][:B], np.float32)
    s = run_case(sh, lp, lq, dtype, T, un, paper_layout=False, pad_to=0, label="dense-unaligned")
    s2 = run_case(sh, lp, lq, dtype, 1.0, un, paper_layout=True, pad_to=8, label="paper-aligned")
    assert s.rows and s2.rows


@pytest.mark.parametrize("split", [0, 8, 1, 2, 4])
@pytest.mark.parametrize("V", [4096, 8192, 9000, 12344, 16384, 16392, 24000, 32768, 40000, 65536, 70000, 81920,
                               131072, 140000, 196608, 200000, 262144, 262152])
def test_lean_shapes(sh, V, split):
    """bf16, aligned, V % 8 == 0: shapes that take the large-vocabulary bf16 kernels (V >= 8192) or, below
    that, the general ones with ragged warp ranges.  split = 8 asks for the exponentials resident on
    chip (1, 2, 4 or 8 CTAs per row and one to four batches per lane, chosen by V; beyond 262144 ids the
    streaming kernels); 1, 2, 4 force the streaming kernels with that many CTAs per row, their loads going
    to registers; 0 is the library's choice: one CTA per row, RRS / RRSw fed by rings of bulk copies."""
    if split not in (0, 8) and V > 81920:
        pytest.skip("the forced-split streaming kernels are covered up to 81920")
    rng = np.random.default_rng(V + 3)
    B, N = 5, 7
    lp, lq = random_logits(rng, B, N, V, "bf16")
    # sprinkle the degenerate kinds in
    lq[0, 1] = lp[0, 1]
    lq[1, 2] = -np.inf; lq[1, 2, V - 1] = 0.0
    lq[2, 0] = -60.0; lq[2, 0, V // 2] = 0.0
    lp[3, 3, : V // 2] = -np.inf; lq[3, 3, V // 2:] = -np.inf
    lp[4, 4] = np.round(lp[4, 4] * 2) / 2; lq[4, 4] = np.round(lq[4, 4] * 2) / 2
    lq[4, 5, 7] = lq[4, 5].max() + 9.0   # peaked draft
    lp, lq = workloads.round_to_storage(lp, "bf16"), workloads.round_to_storage(lq, "bf16")
    un = random_uniforms(rng, B, N)
    T = np.array([1.0, 0.6, 1.3, 0.8, 1.0], np.float32)
    sh.set_row_split(split)
    try:
        run_case(sh, lp, lq, "bf16", T, un, paper_layout=False, label="lean-dense-split%d" % split)
        run_case(sh, lp, lq, "bf16", 1.0, un, paper_layout=True, label="lean-paper-split%d" % split)
    finally:
        sh.set_row_split(0)


@pytest.mark.parametrize("V,dtype", [(1000, "fp32"), (12344, "bf16"), (40000, "bf16")])
def test_low_temperature_large_logits(sh, V, dtype):
    """Logits clustered around 30 at T = 0.1-0.3: k * max logit reaches several hundred, where the
    rounding of that product is 1e-5 and may not leak into the normaliser.  (The cluster is tight so
    that the mass outside the top token stays far above fp32's underflow.)"""
    rng = np.random.default_rng(V + 77)
    B, N = 4, 7
    lp = rng.normal(0, 0.3, (B, N, V)).astype(np.float32) + 30.0
    lq = lp + rng.normal(0, 0.1, (B, N, V)).astype(np.float32)
    lp[:, :, 11] += 0.6; lq[:, :, 11] += 0.6          # a clear top token
    lp, lq = workloads.round_to_storage(lp, dtype), workloads.round_to_storage(lq, dtype)
    un = random_uniforms(rng, B, N)
    T = np.array([0.1, 0.2, 0.3, 1.0], np.float32)
    run_case(sh, lp, lq, dtype, T, un, paper_layout=False, label="low-T")
    run_case(sh, lp, lq, dtype, 0.1, un, paper_layout=True, label="low-T-paper")


@pytest.mark.parametrize("V", [16384, 40000, 131072])
def test_exponent_reference_moves(sh, V):
    """Rows whose first logits lie hundreds of units below the later ones: the running sums leave
    the range of their first exponent reference, in some lanes of a warp and not in others."""
    rng = np.random.default_rng(V + 5)
    B, N = 3, 7
    lp, lq = random_logits(rng, B, N, V, "bf16")
    lq[0, 0, : V // 2] -= 300.0; lp[0, 0, : V // 2] -= 300.0          # low first half, both rows
    lq[0, 1, ::2] -= 250.0                                             # every other id low (lanes differ)
    lp[0, 2, : V // 3] = -np.inf; lp[0, 2, V // 3: V // 2] -= 400.0    # -inf, then low, then normal
    lq[1, 3, :100] += 300.0                                            # a high start, the rest far below
    lq[1, 4, V - 50:] += 280.0; lp[1, 4, V - 50:] += 280.0             # the mass arrives at the very end
    lq[2, 5, 1000:1010] += 200.0
    lp, lq = workloads.round_to_storage(lp, "bf16"), workloads.round_to_storage(lq, "bf16")
    un = random_uniforms(rng, B, N)
    T = np.array([1.0, 0.7, 1.5], np.float32)
    run_case(sh, lp, lq, "bf16", T, un, paper_layout=False, label="moving-reference")
    run_case(sh, lp, lq, "bf16", 1.0, un, paper_layout=True, label="moving-reference-paper")


@pytest.mark.parametrize("V,dtype", [(1000, "fp32"), (12344, "bf16"), (40000, "bf16")])
def test_decisions_without_probabilities(sh, V, dtype):
    """With no beta / rate buffers the library may stop after the first test; decisions, tokens,
    hub and the walk must be the same as with them (bit for bit: same kernels, same arithmetic)."""
    rng = np.random.default_rng(V + 17)
    B, N = 6, 7
    lp, lq = random_logits(rng, B, N, V, dtype, sigma=0.7)
    un = random_uniforms(rng, B, N)
    tp, tq, und = workloads.to_device(lp, dtype), workloads.to_device(lq, dtype), torch.from_numpy(un).cuda()
    for paper in (False, True):
        tree = sh.Tree.heap(N, leaves_sample=paper)
        for m in METHODS:
            d = gpu_draft(sh, m, tq, und, tree, 1.0)
            full = parity.to_numpy(gpu_verify(sh, m, tp, tq, d["tokens"], und, tree, 1.0))
            if m == "spechub":
                lite = sh.spechub_verify_tree(tp, tq, d["tokens"], und, tree, 1.0, probabilities=False)
            else:
                lite = sh.rrs_verify_tree(tp, tq, d["tokens"], und, tree, m == "rrsw", 1.0, probabilities=False)
            lite = parity.to_numpy(lite)
            for k in ("accept_idx", "token", "hub", "n_accepted", "n_emitted", "path_nodes", "path_tokens"):
                np.testing.assert_array_equal(full[k], lite[k], err_msg="%s %s" % (m, k))
            assert (full["accept_idx"] >= 0).any() and (full["accept_idx"] < 0).any()


def test_peaked_rows_keep_precision(sh):
    """q close to one-hot: 1 - q(a) must come from a direct sum, not from 1 - q(a)."""
    rng = np.random.default_rng(5)
    B, N, V = 4, 3, 5000
    lp, lq = random_logits(rng, B, N, V, "fp32")
    for b in range(B):
        lq[b, :, 17 + b] += 12.0 + 4 * b
    un = random_uniforms(rng, B, N)
    un[:, :, 0] = 0.5  # x1 = hub, so the second draw and c = q(a)/(1-q(a)) are exercised
    run_case(sh, lp, lq, "fp32", 1.0, un, paper_layout=False, label="peaked")


# ------------------------------------------------------------------------------------------------
# degenerate and malformed rows
# ------------------------------------------------------------------------------------------------

def test_degenerate_rows(sh):
    rng = np.random.default_rng(11)
    V = 2048
    lp, lq = random_logits(rng, 1, 7, V, "bf16")
    lq[0, 0] = lp[0, 0]                                   # p = q: never rejects
    lq[0, 1] = -np.inf; lq[0, 1, 77] = 0.0                # one-hot q
    lq[0, 2] = -60.0; lq[0, 2, 5] = 0.0                   # nearly one-hot q
    lp[0, 3, :1024] = -np.inf; lq[0, 3, 1024:] = -np.inf  # disjoint supports
    lq[0, 4] = workloads.round_to_storage(rng.normal(0, 0.01, V).astype(np.float32), "bf16")
    lp[0, 5] = np.round(lp[0, 5] * 2) / 2; lq[0, 5] = np.round(lq[0, 5] * 2) / 2  # many exact ties
    lq[0, 6] = 0.0                                        # exactly uniform q: hub = id 0
    for seed in range(4):
        un = random_uniforms(np.random.default_rng(seed), 1, 7)
        run_case(sh, lp, lq, "bf16", 1.0, un, paper_layout=False, label="degenerate")


def test_flagged_rows(sh):
    rng = np.random.default_rng(12)
    V = 1000
    lp, lq = random_logits(rng, 1, 7, V, "fp32")
    lp[0, 0, 3] = np.nan
    lq[0, 1, 9] = np.inf
    lq[0, 2] = -np.inf
    un = random_uniforms(rng, 1, 7)
    tree = sh.Tree.heap(7)
    tp, tq, und = workloads.to_device(lp, "fp32"), workloads.to_device(lq, "fp32"), torch.from_numpy(un).cuda()
    for m in METHODS:
        d = parity.to_numpy(gpu_draft(sh, m, tq, und, tree, 1.0))
        st, od = parity.check_draft(m, lq, 1.0, un, d)
        assert d["status"][0, 1] & 1 and d["status"][0, 2] & 1 and not d["status"][0, 0] & 1
        tok = od["tokens"].copy()
        tok[0, 0] = tok[0, 1] = tok[0, 2] = (1, 2)
        tok[0, 3] = (V, 0)            # out of range
        tok[0, 4] = (-1, 5)
        hub4 = int(np.argmax(lq[0, 5]))
        tok[0, 5] = (hub4, hub4)      # SpecHub: pair holds the hub twice
        out = parity.to_numpy(gpu_verify(sh, m, tp, tq, torch.from_numpy(tok).cuda(), und, tree, 1.0))
        parity.check_verify(m, lp, lq, 1.0, tok, un, None, out)
        assert (out["status"][0, :3] & 1).all()
        assert (out["status"][0, 3:5] & 2).all()
        assert (out["token"][0, :5] == -1).all()
        assert out["n_emitted"][0] == 0


def test_argument_errors(sh):
    import ctypes

    from paper_2411_05289_b200 import binding

    lib = sh.load_library()
    x = torch.zeros((2, 3, 64), dtype=torch.float32, device="cuda")
    d, _ = binding._desc(x, sh.Tree.heap(3), 1.0)
    un = torch.zeros((2, 3, 5), device="cuda")
    tok = torch.zeros((2, 3, 2), dtype=torch.int32, device="cuda")
    vp = ctypes.c_void_p
    call = lambda dd: lib.spechub_draft_sample(ctypes.byref(dd), vp(x.data_ptr()), vp(un.data_ptr()),
                                               vp(tok.data_ptr()), None, None, None, None)
    assert call(d) == 0
    for field, val, code in [("k", 3, -3), ("k", 1, -3), ("vocab", 1, -3), ("dtype", 7, -4), ("version", 9, -2),
                             ("stride_node", 8, -5), ("temperature", 0.0, -6), ("levels", 0, -3),
                             ("flags", 16, -3), ("flags", 3, -3), ("flags", 9, -3)]:
        dd, _ = binding._desc(x, sh.Tree.heap(3), 1.0)
        setattr(dd, field, val)
        assert call(dd) == code, field
    assert lib.spechub_draft_sample(ctypes.byref(d), None, vp(un.data_ptr()), vp(tok.data_ptr()),
                                    None, None, None, None) == -1
    assert lib.rrs_draft_sample(ctypes.byref(d), vp(x.data_ptr()), vp(un.data_ptr()), 2,
                                vp(tok.data_ptr()), None, None) == -9
    torch.cuda.synchronize()
    # empty batch is a no-op
    e = torch.zeros((0, 3, 64), device="cuda")
    out = sh.spechub_draft_sample(e, torch.zeros((0, 3, 5), device="cuda"), sh.Tree.heap(3))
    assert out["tokens"].shape == (0, 3, 2)


@pytest.mark.parametrize("V,dtype", [(1000, "fp32"), (9001, "bf16"), (12344, "bf16"), (40000, "bf16")])
def test_strided_views_equal_contiguous_rows(sh, V, dtype):
    """Rows taken out of a larger buffer (gaps between nodes and between sequences, a base that
    is not the allocation's start) give bit for bit what the same rows give when contiguous."""
    rng = np.random.default_rng(V + 41)
    B, N = 4, 7
    lp, lq = random_logits(rng, B, N, V, dtype)
    un = random_uniforms(rng, B, N)
    und = torch.from_numpy(un).cuda()
    tp, tq = workloads.to_device(lp, dtype), workloads.to_device(lq, dtype)
    Vp = (V + 15) // 16 * 16 + 16

    def embed(t):
        big = torch.full((B + 1, N + 3, Vp), float("nan"), dtype=t.dtype, device="cuda")
        view = big[1:, 2:N + 2, 8:8 + V]
        view.copy_(t)
        return view

    sp, sq = embed(tp), embed(tq)
    assert not sp.is_contiguous() and sp.stride(2) == 1
    tree = sh.Tree.heap(N)
    for m in METHODS:
        d_ref = gpu_draft(sh, m, tq, und, tree, 1.0)
        d_str = gpu_draft(sh, m, sq, und, tree, 1.0)
        assert torch.equal(d_ref["tokens"], d_str["tokens"]) and torch.equal(d_ref["status"], d_str["status"])
        ref = gpu_verify(sh, m, tp, tq, d_ref["tokens"], und, tree, 1.0)
        got = gpu_verify(sh, m, sp, sq, d_ref["tokens"], und, tree, 1.0)
        for k in ref:
            a, b = ref[k], got[k]
            if a.dtype == torch.float32:
                a, b = a.view(torch.int32), b.view(torch.int32)
            assert torch.equal(a, b), "%s %s" % (m, k)
    all3 = sh.mdsd_compare_verify_tree(sp, sq, {m: gpu_draft(sh, m, tq, und, tree, 1.0)["tokens"] for m in METHODS},
                                       und, tree, 1.0)
    ref0 = gpu_verify(sh, "spechub", tp, tq, gpu_draft(sh, "spechub", tq, und, tree, 1.0)["tokens"], und, tree, 1.0)
    assert torch.equal(all3["spechub"]["token"], ref0["token"])


def test_custom_child_table_and_determinism(sh):
    rng = np.random.default_rng(21)
    B, N, V = 16, 5, 3000
    lp, lq = random_logits(rng, B, N, V, "bf16", sigma=0.3)
    un = random_uniforms(rng, B, N)
    child = np.array([[1, 2], [3, -1], [4, -1], [-1, -1], [-1, -1]], np.int32)  # unbalanced tree
    kind = np.array([0, 0, 0, 1, 0], np.uint8)
    tree = sh.Tree(levels=3, child=torch.from_numpy(child).cuda(), node_kind=torch.from_numpy(kind).cuda())
    tp, tq, und = workloads.to_device(lp, "bf16"), workloads.to_device(lq, "bf16"), torch.from_numpy(un).cuda()
    d = gpu_draft(sh, "spechub", tq, und, tree, 1.0)
    o1 = parity.to_numpy(gpu_verify(sh, "spechub", tp, tq, d["tokens"], und, tree, 1.0))
    o2 = parity.to_numpy(gpu_verify(sh, "spechub", tp, tq, d["tokens"], und, tree, 1.0))
    for k in o1:
        np.testing.assert_array_equal(o1[k], o2[k], err_msg=k)  # bit-identical across runs
    w = oracle.walk(o1["accept_idx"], o1["token"], 3, child=child, node_kind=kind)
    for k in ("n_accepted", "n_emitted", "path_nodes", "path_tokens"):
        np.testing.assert_array_equal(o1[k], w[k])
    parity.check_verify("spechub", lp, lq, 1.0, parity.to_numpy(d)["tokens"], un, kind, o1)


# ------------------------------------------------------------------------------------------------
# the benchmark configurations
# ------------------------------------------------------------------------------------------------

def test_config1_full(sh):
    cfg = workloads.CONFIGS["c1"]
    lp, lq = workloads.host_logits(cfg)
    un = workloads.host_uniforms(cfg)
    for paper in (True, False):
        s = run_case(sh, lp, lq, cfg.dtype, cfg.temperature, un, paper_layout=paper, label="c1")
        report("c1 paper=%s" % paper, s)


def test_config2_full(sh):
    cfg = workloads.CONFIGS["c2"]
    lp, lq = workloads.host_logits(cfg)
    un = workloads.host_uniforms(cfg)
    for paper in (False, True):
        s = run_case(sh, lp, lq, cfg.dtype, cfg.temperature, un, paper_layout=paper, label="c2")
        report("c2 paper=%s" % paper, s)


def sampled_parity(sh, cfg, n_sample, layouts=(False,), extra_rows=(), pool=None, with_stats=True):
    """Full-size run on device-generated inputs; oracle (on all host cores) on sampled rows, spread
    evenly over the tree's nodes, plus `extra_rows`.  with_stats: the same rows also through the entry
    points that hand the draft statistics from the draft call to verification."""
    tp, tq = workloads.device_logits(cfg)
    und = workloads.device_uniforms(cfg)
    B, N, V = tp.shape
    rng = np.random.default_rng(cfg.seed + 99)
    # the same number of rows from every node of the tree (every level, leaves and inner nodes alike)
    per_node = max(1, min(B, -(-n_sample // N)))
    rows = sorted(set(int(b) * N + n for n in range(N) for b in rng.choice(B, size=per_node, replace=False))
                  | set(extra_rows))
    bs, ns = np.array([r // N for r in rows]), np.array([r % N for r in rows])
    idx_b, idx_n = torch.from_numpy(bs).cuda(), torch.from_numpy(ns).cuda()
    lp = workloads.to_host_f32(tp[idx_b, idx_n])[:, None, :]
    lq = workloads.to_host_f32(tq[idx_b, idx_n])[:, None, :]
    un = und[idx_b, idx_n].cpu().numpy()[:, None, :]
    total = parity.Stats()
    for paper in layouts:
        tree = sh.Tree.heap(N, leaves_sample=paper)
        kind = workloads.paper_node_kind(N) if paper else None
        for m in METHODS:
            d = gpu_draft(sh, m, tq, und, tree, cfg.temperature)
            out = gpu_verify(sh, m, tp, tq, d["tokens"], und, tree, cfg.temperature)
            torch.cuda.synchronize()
            dn = {k: v[idx_b, idx_n].cpu().numpy()[:, None] for k, v in d.items()}
            st, _ = parity.check_draft(m, lq, cfg.temperature, un, dn, label=cfg.name, pool=pool)
            tok = dn["tokens"]
            on = {k: out[k][idx_b, idx_n].cpu().numpy()[:, None] for k in
                  ("accept_idx", "token", "hub", "beta", "rate", "status")}
            records = {}   # the oracle's records of the sampled rows, kept for the second leg below

            def check_rows(on, label, sv):
                if kind is None:
                    _, records[-1] = parity.check_verify(m, lp, lq, cfg.temperature, tok, un, None, on, stats=sv,
                                                         label=label, pool=pool, oracle_out=records.get(-1))
                    return
                for leafness in (0, 1):
                    sel = np.nonzero(kind[ns] == leafness)[0]
                    if len(sel) == 0:
                        continue
                    sub = {k: v[sel] for k, v in on.items()}
                    _, records[leafness] = parity.check_verify(
                        m, lp[sel], lq[sel], cfg.temperature, tok[sel], un[sel], np.array([leafness], np.uint8), sub,
                        stats=sv, label=label, pool=pool, oracle_out=records.get(leafness))

            sv = parity.Stats()
            check_rows(on, cfg.name, sv)
            if with_stats:
                # the step as bench.py runs it by default: the draft call hands its statistics of the draft rows
                # to verification.  Same drafts (bit for bit), same oracle records, same bar.
                d2 = gpu_draft_stats(sh, m, tq, und, tree, cfg.temperature)
                assert torch.equal(d2["tokens"], d["tokens"])
                out2 = gpu_verify_stats(sh, m, tp, tq, d2["stats"], d2["tokens"], und, tree, cfg.temperature)
                torch.cuda.synchronize()
                assert int((out2["status"] & 3).sum()) == 0 and int((out2["status"] & (32 | 64)).sum()) == 0
                assert float((out2["rate"].sum(-1) - 1).abs().max()) < 1e-4
                on2 = {k: out2[k][idx_b, idx_n].cpu().numpy()[:, None] for k in
                       ("accept_idx", "token", "hub", "beta", "rate", "status")}
                check_rows(on2, cfg.name + "+stats", sv)
                full2 = parity.to_numpy({k: out2[k] for k in ("accept_idx", "token", "n_accepted", "n_emitted",
                                                              "path_nodes", "path_tokens")})
                w2 = oracle.walk(full2["accept_idx"], full2["token"], tree.levels, node_kind=kind)
                for k in ("n_accepted", "n_emitted", "path_nodes", "path_tokens"):
                    np.testing.assert_array_equal(full2[k], w2[k], err_msg=k + " (+stats)")
                del d2, out2
            # the walk, for every sequence, against the oracle's walk of the GPU's node outputs
            full = parity.to_numpy({k: out[k] for k in ("accept_idx", "token", "n_accepted", "n_emitted",
                                                        "path_nodes", "path_tokens")})
            w = oracle.walk(full["accept_idx"], full["token"], tree.levels, node_kind=kind)
            for k in ("n_accepted", "n_emitted", "path_nodes", "path_tokens"):
                np.testing.assert_array_equal(full[k], w[k], err_msg=k)
            # properties that hold at any size
            st_all = out["status"]
            assert int((st_all & 3).sum()) == 0
            assert bool(((out["token"] >= 0) & (out["token"] < V)).all())
            rate = out["rate"]
            assert float((rate.sum(-1) - 1).abs().max()) < 1e-4
            total.add(st).add(sv)
            del d, out
    del tp, tq
    torch.cuda.empty_cache()
    return total


@pytest.mark.parametrize("variant", range(4))
def test_config3_sampled(sh, pool, variant):
    cfg = workloads.variants("c3")[variant]
    s = sampled_parity(sh, cfg, 1024, layouts=(False, True), pool=pool)
    report(cfg.name, s)


@pytest.mark.parametrize("split,n_sample", [(0, 4096), (8, 512), (4, 128)])
def test_config4_sampled(sh, pool, split, n_sample):
    """The default path on 1024+ rows per method and layout; the forced-split streaming kernels on fewer."""
    cfg = workloads.CONFIGS["c4"]
    sh.set_row_split(split)
    try:
        s = sampled_parity(sh, cfg, n_sample, layouts=(False, True), pool=pool, with_stats=(split == 0))
    finally:
        sh.set_row_split(0)
    report("c4 split=%d" % split, s)


def test_config5_sampled(sh, pool):
    cfg = workloads.CONFIGS["c5"]
    if torch.cuda.get_device_properties(0).total_memory < 60e9:
        pytest.skip("needs ~25 GB of device memory")
    # make sure every adversarial kind is among the checked rows
    per_kind = {}
    for b in range(cfg.batch):
        for n in range(cfg.nodes):
            k = workloads._adversarial_kind(cfg, b, n)
            if k >= 0 and len(per_kind.setdefault(k, [])) < 24:
                per_kind[k].append(b * cfg.nodes + n)
    assert len(per_kind) == len(workloads.ADV_KINDS)
    extra = [(r, k) for k, rows in per_kind.items() for r in rows]
    s = sampled_parity(sh, cfg, 2048, extra_rows=[e[0] for e in extra], pool=pool)
    report("c5", s)


# ------------------------------------------------------------------------------------------------
# extremes of the shape: very long rows, very many rows
# ------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("V,dtype", [(1 << 20, "bf16"), ((1 << 20) + 3, "bf16"), (600_001, "fp32")])
def test_very_long_rows(sh, V, dtype):
    """A million-token vocabulary: index arithmetic and the two-level samplers at their far end."""
    rng = np.random.default_rng(V % 1000)
    lp, lq = random_logits(rng, 1, 3, V, dtype, sd=3.0)
    lq[0, 1, V - 1] = lq[0, 1].max() + 4.0        # hub is the very last id
    lp, lq = workloads.round_to_storage(lp, dtype), workloads.round_to_storage(lq, dtype)
    un = random_uniforms(rng, 1, 3)
    un[0, 2, 0] = np.float32(1.0 - 2.0 ** -24)    # the largest uniform: the draw lands at the end of the CDF
    run_case(sh, lp, lq, dtype, 1.0, un, paper_layout=False, label="long-rows")


def test_very_many_rows(sh):
    """More rows than a 16-bit grid dimension holds; a sample of them against the oracle."""
    rng = np.random.default_rng(9)
    B, N, V = 70_001, 1, 24
    lp, lq = random_logits(rng, B, N, V, "fp32")
    un = random_uniforms(rng, B, N)
    tp, tq, und = workloads.to_device(lp, "fp32"), workloads.to_device(lq, "fp32"), torch.from_numpy(un).cuda()
    tree = sh.Tree.heap(1)
    pick = np.unique(np.concatenate([[0, 65535, 65536, B - 1], rng.integers(0, B, 200)]))
    for m in METHODS:
        d = parity.to_numpy(gpu_draft(sh, m, tq, und, tree, 1.0))
        dsub = {k: (v[pick] if v is not None else None) for k, v in d.items()}
        _, od = parity.check_draft(m, lq[pick], 1.0, un[pick], dsub, label="many-rows")
        out = parity.to_numpy(gpu_verify(sh, m, tp, tq, torch.from_numpy(d["tokens"]).cuda(), und, tree, 1.0))
        osub = {k: v[pick] for k, v in out.items()}
        parity.check_verify(m, lp[pick], lq[pick], 1.0, d["tokens"][pick], un[pick], None, osub, label="many-rows")
        w = oracle.walk(out["accept_idx"], out["token"], 1)
        for k in ("n_accepted", "n_emitted", "path_nodes", "path_tokens"):
            np.testing.assert_array_equal(out[k], w[k], err_msg="many-rows walk %s" % k)


def test_calls_on_two_streams_do_not_interfere(sh):
    """The library keeps no state: calls enqueued on two streams, interleaved, give what the same
    calls give one after another."""
    rng = np.random.default_rng(21)
    cases = []
    for V, dtype in ((12344, "bf16"), (5000, "fp32")):
        lp, lq = random_logits(rng, 6, 7, V, dtype)
        un = random_uniforms(rng, 6, 7)
        cases.append((workloads.to_device(lp, dtype), workloads.to_device(lq, dtype), torch.from_numpy(un).cuda()))
    tree = sh.Tree.heap(7)
    ref = []
    for tp, tq, und in cases:
        d = sh.spechub_draft_sample(tq, und, tree, 1.0)
        ref.append((d, sh.spechub_verify_tree(tp, tq, d["tokens"], und, tree, 1.0)))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    got = [None, None]
    for rep in range(3):
        for i, (tp, tq, und) in enumerate(cases):
            with torch.cuda.stream(streams[i]):
                d = sh.spechub_draft_sample(tq, und, tree, 1.0)
                got[i] = (d, sh.spechub_verify_tree(tp, tq, d["tokens"], und, tree, 1.0))
    torch.cuda.synchronize()
    for (dr, vr), (dg, vg) in zip(ref, got):
        assert torch.equal(dr["tokens"], dg["tokens"])
        for k in vr:
            a, b = vr[k], vg[k]
            if a.dtype == torch.float32:
                a, b = a.view(torch.int32), b.view(torch.int32)
            assert torch.equal(a, b), k


def test_unbalanced_tree_from_parents(sh):
    """A binary tree with missing children (the shape of the paper's unbalanced Sequoia trees):
    childless nodes draw the bonus token, the walk follows the child table."""
    parents = [-1, 0, 0, 1, 1, 2, 3, 3, 4, 6]
    tree = sh.Tree.from_parents(parents)
    child = tree.child.cpu().numpy()
    kind = tree.node_kind.cpu().numpy()
    N = len(parents)
    rng = np.random.default_rng(31)
    for V, dtype in ((9000, "bf16"), (777, "fp32")):
        B = 6
        lp, lq = random_logits(rng, B, N, V, dtype, sigma=0.6)
        un = random_uniforms(rng, B, N)
        tp, tq, und = workloads.to_device(lp, dtype), workloads.to_device(lq, dtype), torch.from_numpy(un).cuda()
        for m in METHODS:
            d = parity.to_numpy(gpu_draft(sh, m, tq, und, tree, 1.0))
            _, od = parity.check_draft(m, lq, 1.0, un, d, label="unbalanced")
            tok = od["tokens"].copy()
            out = parity.to_numpy(gpu_verify(sh, m, tp, tq, torch.from_numpy(tok).cuda(), und, tree, 1.0))
            parity.check_verify(m, lp, lq, 1.0, tok, un, kind, out, label="unbalanced")
            w = oracle.walk(out["accept_idx"], out["token"], tree.levels, child=child, node_kind=kind)
            for k in ("n_accepted", "n_emitted", "path_nodes", "path_tokens"):
                np.testing.assert_array_equal(out[k], w[k], err_msg="unbalanced walk %s" % k)
            assert out["n_accepted"].max() >= 2


def test_walk_stops_at_an_accept_index_outside_the_children(sh):
    """spechub_walk_tree takes a caller-supplied accept_idx (the vocabulary-sharded path hands it the
    exchanged array): an index that names no child ends the walk at that node instead of indexing
    past the child table."""
    import ctypes

    from paper_2411_05289_b200 import binding, vocab_sharded

    lib = vocab_sharded._lib()
    B, N = 3, 7
    tree = sh.Tree.heap(N)
    x = torch.zeros((B, N, 64), dtype=torch.float32, device="cuda")
    d, _ = binding._desc(x, tree, 1.0)
    acc = torch.tensor([[0, 2, 0, 0, 0, 0, 0], [1, 0, 2147483647, 0, 0, 0, 0], [0, 1, 0, 0, 0, 0, 0]],
                       dtype=torch.int32, device="cuda")
    tok = torch.arange(B * N, dtype=torch.int32, device="cuda").reshape(B, N) + 100
    out = binding.alloc_verify_outputs(B, N, tree.levels, x.device)
    so = binding._SeqOut(*[out[k].data_ptr() for k in ("n_accepted", "n_emitted", "path_nodes", "path_tokens")])
    rc = lib.spechub_walk_tree(ctypes.byref(d), ctypes.c_void_p(acc.data_ptr()), ctypes.c_void_p(tok.data_ptr()),
                               ctypes.byref(so), None)
    assert rc == 0
    torch.cuda.synchronize()
    assert out["path_nodes"].cpu().tolist() == [[0, 1, -1], [0, 2, -1], [0, 1, 4]]
    assert out["n_accepted"].cpu().tolist() == [1, 1, 3]
    assert out["n_emitted"].cpu().tolist() == [2, 2, 3]
