"""The law of the emitted token on the GPU path itself (Theorem 2 for SpecHub; Algorithm 1's
guarantee for RRS / RRSw): many rows with the same (p, q) and independent uniforms; the token that
comes out of draft + verification must be distributed as p, and the branches must be taken as
often as the kernels' own `rate` outputs say.  No oracle value is involved."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def sh():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2411_05289_b200 as lib

    lib.load_library()
    return lib


def chi2_ok(counts, probs, n):
    from scipy.stats import chi2

    keep = probs * n >= 5
    stat = float((((counts - probs * n) ** 2) / (probs * n))[keep].sum())
    return chi2.sf(stat, int(keep.sum()) - 1) > 1e-5, stat


@pytest.mark.parametrize("method", ["spechub", "rrs", "rrsw"])
@pytest.mark.parametrize("V,T,seed", [(12, 1.0, 1), (50, 0.6, 2), (9000, 1.0, 3)])
def test_emitted_token_follows_the_target(sh, method, V, T, seed):
    n = 200_000 if V < 1000 else 60_000
    g = torch.Generator(device="cuda").manual_seed(seed)
    sd = 1.5 if V < 1000 else 3.0
    lp = torch.randn(V, device="cuda", generator=g) * sd
    lq = lp + torch.randn(V, device="cuda", generator=g) * 0.8
    dtype = torch.float32 if V < 1000 else torch.bfloat16
    lp, lq = lp.to(dtype), lq.to(dtype)
    tp = lp.expand(n, 1, V).contiguous()
    tq = lq.expand(n, 1, V).contiguous()
    un = torch.rand((n, 1, 5), device="cuda", generator=g)
    tree = sh.Tree.heap(1)
    if method == "spechub":
        d = sh.spechub_draft_sample(tq, un, tree, T)
        out = sh.spechub_verify_tree(tp, tq, d["tokens"], un, tree, T)
    else:
        wo = method == "rrsw"
        d = sh.rrs_draft_sample(tq, un, tree, wo, T)
        out = sh.rrs_verify_tree(tp, tq, d["tokens"], un, tree, wo, T)
    torch.cuda.synchronize()
    assert int(out["status"].bitwise_and(3).sum()) == 0
    p = torch.softmax(lp.double() / T, 0).cpu().numpy()
    q = torch.softmax(lq.double() / T, 0).cpu().numpy()
    tok = out["token"].view(-1).cpu().numpy()
    ok, stat = chi2_ok(np.bincount(tok, minlength=V).astype(np.float64), p, n)
    assert ok, "emitted tokens do not follow p (chi2 = %.1f)" % stat
    # the first draft follows q
    ok, stat = chi2_ok(np.bincount(d["tokens"][:, 0, 0].cpu().numpy(), minlength=V).astype(np.float64), q, n)
    assert ok, "x1 does not follow q (chi2 = %.1f)" % stat
    # branches are taken as often as the reported rates say (RRSw's later rates are conditional on
    # the given x1 being the rejected one, so only its first rate is an unconditional frequency)
    acc = out["accept_idx"].view(-1).cpu().numpy()
    rate = out["rate"].view(n, 3).double().cpu().numpy()
    checks = [(acc == 0).mean() - rate[:, 0].mean()]
    if method != "rrsw":
        checks += [(acc == 1).mean() - rate[:, 1].mean(), (acc < 0).mean() - rate[:, 2].mean()]
    for c in checks:
        assert abs(c) < 5 * 0.5 / np.sqrt(n), checks
