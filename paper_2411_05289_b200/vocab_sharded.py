"""SpecHub over a vocabulary-sharded LM head: one rank per slice of token ids.

Each rank calls the phases of ``include/spechub.h`` ("vocabulary axis sharded over ranks") on its
own slice and exchanges a few floats per row between them.  ``ShardedDraft`` / ``ShardedVerify``
hold one rank's state and expose the phases one by one, so that a driver can run ranks in lockstep;
``spechub_draft_sample_sharded`` / ``spechub_verify_tree_sharded`` are that driver for
``torch.distributed`` (one process per GPU, NCCL): two small all-gathers and one element-wise
maximum per call.  Argument marshalling and collectives only; all arithmetic is in the kernels.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass

import torch

from . import binding as _b


class _Shard(ctypes.Structure):
    _fields_ = [("rank", ctypes.c_int32), ("nranks", ctypes.c_int32), ("id_offset", ctypes.c_int32),
                ("vocab_total", ctypes.c_int32)]


@dataclass(frozen=True)
class Shard:
    rank: int
    nranks: int
    id_offset: int
    vocab_total: int

    def c(self):
        return _Shard(self.rank, self.nranks, self.id_offset, self.vocab_total)


def even_shards(vocab_total: int, nranks: int):
    """Contiguous id ranges, the first `vocab_total % nranks` one token wider."""
    out, off = [], 0
    for r in range(nranks):
        w = vocab_total // nranks + (1 if r < vocab_total % nranks else 0)
        out.append((Shard(r, nranks, off, vocab_total), w))
        off += w
    return out


_configured = False


def _lib():
    global _configured
    lib = _b.load_library()
    if not _configured:
        vp, i32 = ctypes.c_void_p, ctypes.c_int
        D, S = ctypes.POINTER(_b._Desc), ctypes.POINTER(_Shard)
        lib.spechub_walk_tree.restype = i32
        lib.spechub_walk_tree.argtypes = [D, vp, vp, ctypes.POINTER(_b._SeqOut), vp]
        lib.spechub_shard_stats.restype = i32
        lib.spechub_shard_stats.argtypes = [D, S, vp, vp, vp, vp]
        lib.spechub_shard_sums.restype = i32
        lib.spechub_shard_sums.argtypes = [D, S, vp, vp, vp, vp, vp, vp]
        lib.spechub_shard_decide.restype = i32
        lib.spechub_shard_decide.argtypes = [D, S, vp, vp, vp, vp, vp, vp, ctypes.POINTER(_b._NodeOut), vp]
        lib.spechub_shard_draft.restype = i32
        lib.spechub_shard_draft.argtypes = [D, S, vp, vp, vp, vp, vp]
        lib.spechub_shard_draft_finish.restype = i32
        lib.spechub_shard_draft_finish.argtypes = [D, S, vp, vp, vp, vp, vp, vp]
        lib.rrs_shard_sums.restype = i32
        lib.rrs_shard_sums.argtypes = [D, S, i32, vp, vp, vp, vp, vp, vp, vp]
        lib.rrs_shard_decide.restype = i32
        lib.rrs_shard_decide.argtypes = [D, S, i32, vp, vp, vp, vp, vp, vp, vp, ctypes.POINTER(_b._NodeOut), vp]
        lib.rrs_shard_draft.restype = i32
        lib.rrs_shard_draft.argtypes = [D, S, i32, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.rrs_shard_draft_finish.restype = i32
        lib.rrs_shard_draft_finish.argtypes = [D, S, i32, vp, vp, vp, vp, vp]
        _configured = True
    return lib


def _gathered_ok(t, shard, B, N):
    if (t.dtype != torch.float32 or tuple(t.shape) != (shard.nranks, B, N, 8) or not t.is_contiguous()):
        raise ValueError("gathered phase outputs must be contiguous float32 [nranks][batch][nodes][8]")


class _Phases:
    def __init__(self, slice_for_desc, shard: Shard, tree: _b.Tree, temperature, uniforms, stream):
        _b._need_k2(tree)
        self.lib = _lib()
        self.shard, self.cshard = shard, shard.c()
        self.tree = tree
        self.desc, self._keep = _b._desc(slice_for_desc, tree, temperature)
        self.B, self.N, self.width = slice_for_desc.shape
        self.dev = slice_for_desc.device
        _b._check_uniforms(uniforms, self.B, self.N, self.dev)
        self.uniforms = uniforms
        self.stream = stream

    def _new(self, shape, dtype):
        return torch.empty(shape, dtype=dtype, device=self.dev)

    def _sp(self):
        return _b._stream_ptr(self.stream)


class ShardedDraft(_Phases):
    """One rank's side of the draft step."""

    def __init__(self, draft_slice, uniforms, tree, shard, temperature=1.0, stream=None):
        super().__init__(draft_slice, shard, tree, temperature, uniforms, stream)
        self.draft = draft_slice

    def stats(self):
        out = self._new((self.B, self.N, 8), torch.float32)
        _b._check(self.lib.spechub_shard_stats(ctypes.byref(self.desc), ctypes.byref(self.cshard), None,
                                               _b._ptr(self.draft), _b._ptr(out), self._sp()))
        return out

    def candidates(self, gathered_stats):
        _gathered_ok(gathered_stats, self.shard, self.B, self.N)
        self.gstats = gathered_stats
        cand = self._new((self.B, self.N, 2), torch.int32)
        _b._check(self.lib.spechub_shard_draft(ctypes.byref(self.desc), ctypes.byref(self.cshard),
                                               _b._ptr(self.draft), _b._ptr(self.uniforms),
                                               _b._ptr(gathered_stats), _b._ptr(cand), self._sp()))
        return cand

    def finish(self, cand_max):
        tokens = self._new((self.B, self.N, 2), torch.int32)
        hub = self._new((self.B, self.N), torch.int32)
        status = self._new((self.B, self.N), torch.int32)
        _b._check(self.lib.spechub_shard_draft_finish(ctypes.byref(self.desc), ctypes.byref(self.cshard),
                                                      _b._ptr(self.gstats), _b._ptr(cand_max.contiguous()),
                                                      _b._ptr(tokens), _b._ptr(hub), _b._ptr(status), self._sp()))
        return dict(tokens=tokens, hub=hub, status=status)


class ShardedVerify(_Phases):
    """One rank's side of verification and the tree walk."""

    def __init__(self, target_slice, draft_slice, draft_tokens, uniforms, tree, shard, temperature=1.0,
                 stream=None):
        _b._same_layout(target_slice, draft_slice)
        super().__init__(target_slice, shard, tree, temperature, uniforms, stream)
        if (draft_tokens.dtype != torch.int32 or tuple(draft_tokens.shape) != (self.B, self.N, 2)
                or not draft_tokens.is_contiguous()):
            raise ValueError("draft_tokens must be a contiguous int32 [batch][nodes][2] tensor")
        self.target, self.draft, self.tokens = target_slice, draft_slice, draft_tokens

    def stats(self):
        out = self._new((self.B, self.N, 8), torch.float32)
        _b._check(self.lib.spechub_shard_stats(ctypes.byref(self.desc), ctypes.byref(self.cshard),
                                               _b._ptr(self.target), _b._ptr(self.draft), _b._ptr(out), self._sp()))
        return out

    def sums(self, gathered_stats):
        _gathered_ok(gathered_stats, self.shard, self.B, self.N)
        self.gstats = gathered_stats
        out = self._new((self.B, self.N, 8), torch.float32)
        _b._check(self.lib.spechub_shard_sums(ctypes.byref(self.desc), ctypes.byref(self.cshard),
                                              _b._ptr(self.target), _b._ptr(self.draft), _b._ptr(self.tokens),
                                              _b._ptr(gathered_stats), _b._ptr(out), self._sp()))
        return out

    def decide(self, gathered_sums):
        _gathered_ok(gathered_sums, self.shard, self.B, self.N)
        self.out = _b.alloc_verify_outputs(self.B, self.N, self.tree.levels, self.dev)
        no = _b._NodeOut(*[self.out[k].data_ptr() for k in ("accept_idx", "token", "hub", "beta", "rate", "status")])
        _b._check(self.lib.spechub_shard_decide(ctypes.byref(self.desc), ctypes.byref(self.cshard),
                                                _b._ptr(self.target), _b._ptr(self.draft), _b._ptr(self.tokens),
                                                _b._ptr(self.uniforms), _b._ptr(self.gstats),
                                                _b._ptr(gathered_sums), ctypes.byref(no), self._sp()))
        return self.out["token"]

    def walk(self, token_max):
        self.out["token"] = token_max.contiguous()
        so = _b._SeqOut(*[self.out[k].data_ptr() for k in ("n_accepted", "n_emitted", "path_nodes", "path_tokens")])
        _b._check(self.lib.spechub_walk_tree(ctypes.byref(self.desc), _b._ptr(self.out["accept_idx"]),
                                             _b._ptr(self.out["token"]), ctypes.byref(so), self._sp()))
        return self.out


class ShardedRrsDraft(ShardedDraft):
    """One rank's side of the RRS / RRSw draft step (RRSw takes a second round: `second`)."""

    def __init__(self, draft_slice, uniforms, tree, shard, without_replacement, temperature=1.0, stream=None):
        super().__init__(draft_slice, uniforms, tree, shard, temperature, stream)
        self.wo = int(bool(without_replacement))

    def candidates(self, gathered_stats):
        """-> (cand [B][N][2] int32, ex1 [B][N] float32); take the maximum of both over ranks."""
        _gathered_ok(gathered_stats, self.shard, self.B, self.N)
        self.gstats = gathered_stats
        cand = self._new((self.B, self.N, 2), torch.int32)
        ex1 = self._new((self.B, self.N), torch.float32)
        _b._check(self.lib.rrs_shard_draft(ctypes.byref(self.desc), ctypes.byref(self.cshard), self.wo,
                                           _b._ptr(self.draft), _b._ptr(self.uniforms), _b._ptr(gathered_stats),
                                           None, None, _b._ptr(cand), _b._ptr(ex1), self._sp()))
        return cand, ex1

    def second(self, cand_max, ex1_max):
        """RRSw: x2 ~ q without x1 -> cand [B][N][2]; take the maximum over ranks again."""
        cand = self._new((self.B, self.N, 2), torch.int32)
        _b._check(self.lib.rrs_shard_draft(ctypes.byref(self.desc), ctypes.byref(self.cshard), self.wo,
                                           _b._ptr(self.draft), _b._ptr(self.uniforms), _b._ptr(self.gstats),
                                           _b._ptr(cand_max.contiguous()), _b._ptr(ex1_max.contiguous()),
                                           _b._ptr(cand), None, self._sp()))
        return cand

    def finish(self, cand_max):
        tokens = self._new((self.B, self.N, 2), torch.int32)
        status = self._new((self.B, self.N), torch.int32)
        _b._check(self.lib.rrs_shard_draft_finish(ctypes.byref(self.desc), ctypes.byref(self.cshard), self.wo,
                                                  _b._ptr(self.gstats), _b._ptr(cand_max.contiguous()),
                                                  _b._ptr(tokens), _b._ptr(status), self._sp()))
        return dict(tokens=tokens, status=status)


class ShardedRrsVerify(ShardedVerify):
    """One rank's side of RRS / RRSw verification: stats, sums, w2, decide, walk."""

    def __init__(self, target_slice, draft_slice, draft_tokens, uniforms, tree, shard, without_replacement,
                 temperature=1.0, stream=None):
        super().__init__(target_slice, draft_slice, draft_tokens, uniforms, tree, shard, temperature, stream)
        self.wo = int(bool(without_replacement))

    def _sums(self, gathered_sums):
        out = self._new((self.B, self.N, 8), torch.float32)
        _b._check(self.lib.rrs_shard_sums(ctypes.byref(self.desc), ctypes.byref(self.cshard), self.wo,
                                          _b._ptr(self.target), _b._ptr(self.draft), _b._ptr(self.tokens),
                                          _b._ptr(self.gstats), _b._ptr(gathered_sums), _b._ptr(out), self._sp()))
        return out

    def sums(self, gathered_stats):
        _gathered_ok(gathered_stats, self.shard, self.B, self.N)
        self.gstats = gathered_stats
        return self._sums(None)

    def w2(self, gathered_sums):
        _gathered_ok(gathered_sums, self.shard, self.B, self.N)
        self.gsums = gathered_sums
        return self._sums(gathered_sums)

    def decide(self, gathered_w2):
        _gathered_ok(gathered_w2, self.shard, self.B, self.N)
        self.out = _b.alloc_verify_outputs(self.B, self.N, self.tree.levels, self.dev)
        no = _b._NodeOut(*[self.out[k].data_ptr() for k in ("accept_idx", "token", "hub", "beta", "rate", "status")])
        _b._check(self.lib.rrs_shard_decide(ctypes.byref(self.desc), ctypes.byref(self.cshard), self.wo,
                                            _b._ptr(self.target), _b._ptr(self.draft), _b._ptr(self.tokens),
                                            _b._ptr(self.uniforms), _b._ptr(self.gstats), _b._ptr(self.gsums),
                                            _b._ptr(gathered_w2), ctypes.byref(no), self._sp()))
        return self.out["token"]


# ---- the collectives -----------------------------------------------------------------------------

def all_gather_ranks(t, group=None):
    """[...] on every rank -> [nranks][...] in rank order."""
    import torch.distributed as dist

    n = dist.get_world_size(group)
    out = torch.empty((n,) + tuple(t.shape), dtype=t.dtype, device=t.device)
    dist.all_gather(list(out.unbind(0)), t.contiguous(), group=group)  # views: lands in `out` directly
    return out


def all_max(t, group=None):
    import torch.distributed as dist

    t = t.clone()
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return t


def shard_of_group(width: int, group=None) -> Shard:
    """This rank's Shard when every rank tells its slice width (one small all-gather on the host)."""
    import torch.distributed as dist

    n, r = dist.get_world_size(group), dist.get_rank(group)
    widths = [None] * n
    dist.all_gather_object(widths, int(width), group=group)
    return Shard(r, n, sum(widths[:r]), sum(widths))


def slice_of_rank(logits, rank: int, nranks: int):
    """This rank's share of full-vocabulary logits [B][N][V] (a tensor-parallel LM head would hand
    every rank exactly this): the Shard of ``even_shards`` and a contiguous copy of its id range, so
    that each rank's kernels read its own memory only.  Slices are 16-byte aligned when the width is
    a multiple of 8 bf16 ids."""
    V = logits.shape[-1]
    shard, width = even_shards(V, nranks)[rank]
    return shard, logits[..., shard.id_offset:shard.id_offset + width].contiguous()


def _on(stream):
    """The drivers below mix kernel launches, allocations and collectives; all of them follow torch's
    current stream, so a caller's stream is made current for the whole call (kernels launched on one
    stream and collectives on another would race)."""
    import contextlib

    return contextlib.nullcontext() if stream is None else torch.cuda.stream(stream)


def spechub_draft_sample_sharded(draft_slice, uniforms, tree, shard: Shard, temperature=1.0, group=None,
                                 stream=None):
    with _on(stream):
        d = ShardedDraft(draft_slice, uniforms, tree, shard, temperature, None)
        cand = d.candidates(all_gather_ranks(d.stats(), group))
        return d.finish(all_max(cand, group))


def spechub_verify_tree_sharded(target_slice, draft_slice, draft_tokens, uniforms, tree, shard: Shard,
                                temperature=1.0, group=None, stream=None):
    with _on(stream):
        v = ShardedVerify(target_slice, draft_slice, draft_tokens, uniforms, tree, shard, temperature, None)
        gsums = all_gather_ranks(v.sums(all_gather_ranks(v.stats(), group)), group)
        return v.walk(all_max(v.decide(gsums), group))


def rrs_draft_sample_sharded(draft_slice, uniforms, tree, shard: Shard, without_replacement, temperature=1.0,
                             group=None, stream=None):
    with _on(stream):
        d = ShardedRrsDraft(draft_slice, uniforms, tree, shard, without_replacement, temperature, None)
        cand, ex1 = d.candidates(all_gather_ranks(d.stats(), group))
        cand, ex1 = all_max(cand, group), all_max(ex1, group)
        if without_replacement:
            cand = all_max(d.second(cand, ex1), group)
        return d.finish(cand)


def rrs_verify_tree_sharded(target_slice, draft_slice, draft_tokens, uniforms, tree, shard: Shard,
                            without_replacement, temperature=1.0, group=None, stream=None):
    with _on(stream):
        v = ShardedRrsVerify(target_slice, draft_slice, draft_tokens, uniforms, tree, shard, without_replacement,
                             temperature, None)
        gsums = all_gather_ranks(v.sums(all_gather_ranks(v.stats(), group)), group)
        gw2 = all_gather_ranks(v.w2(gsums), group)
        return v.walk(all_max(v.decide(gw2), group))
