"""ctypes binding of ``libspechub.so``: argument marshalling only.

Function names and argument meaning follow ``include/spechub.h``.  Tensors are
torch CUDA tensors; outputs are allocated here with torch (device memory is the
only thing torch is used for) and returned in small dicts.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

from . import build as _build

ABI_VERSION = 1
F32, BF16 = 0, 1

STATUS_BITS = {
    "NONFINITE": 1,
    "TOKEN_RANGE": 2,
    "DEGENERATE_Q": 4,
    "ZERO_MASS_DRAFT": 8,
    "ZERO_RESIDUAL": 16,
    "INTERNAL": 32,
    "STATS": 64,
}


class SpecHubError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__("spechub error %d: %s" % (code, msg))
        self.code = code


class _Desc(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("version", ctypes.c_uint32),
        ("batch", ctypes.c_int32),
        ("nodes", ctypes.c_int32),
        ("vocab", ctypes.c_int32),
        ("k", ctypes.c_int32),
        ("dtype", ctypes.c_int32),
        ("levels", ctypes.c_int32),
        ("stride_seq", ctypes.c_int64),
        ("stride_node", ctypes.c_int64),
        ("temperature", ctypes.c_float),
        ("temperature_per_seq", ctypes.c_void_p),
        ("child", ctypes.c_void_p),
        ("node_kind", ctypes.c_void_p),
        ("flags", ctypes.c_uint32),
    ]


class _NodeOut(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("accept_idx", "token", "hub", "beta", "rate", "status")]


class _SeqOut(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("n_accepted", "n_emitted", "path_nodes", "path_tokens")]


_lib = None


def library_path() -> str:
    return _build.LIB_PATH


def load_library(build_if_missing: bool = True):
    """Load ``libspechub.so`` (building it with nvcc when it is missing or stale).

    Raises if the library cannot be produced: there is no other implementation to fall back to.
    """
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if build_if_missing and _build.is_stale():
        path = _build.build_library()
    if not os.path.exists(path):
        raise SpecHubError(-100, "CUDA library %s is missing; run paper_2411_05289_b200.build" % path)
    lib = ctypes.CDLL(path)
    vp, i32 = ctypes.c_void_p, ctypes.c_int
    lib.spechub_draft_sample.restype = i32
    lib.spechub_draft_sample.argtypes = [ctypes.POINTER(_Desc), vp, vp, vp, vp, vp, vp, vp]
    lib.rrs_draft_sample.restype = i32
    lib.rrs_draft_sample.argtypes = [ctypes.POINTER(_Desc), vp, vp, i32, vp, vp, vp]
    lib.spechub_verify_tree.restype = i32
    lib.spechub_verify_tree.argtypes = [ctypes.POINTER(_Desc), vp, vp, vp, vp,
                                        ctypes.POINTER(_NodeOut), ctypes.POINTER(_SeqOut), vp,
                                        ctypes.c_size_t, vp]
    lib.rrs_verify_tree.restype = i32
    lib.rrs_verify_tree.argtypes = [ctypes.POINTER(_Desc), vp, vp, vp, vp, i32,
                                    ctypes.POINTER(_NodeOut), ctypes.POINTER(_SeqOut), vp,
                                    ctypes.c_size_t, vp]
    lib.spechub_draft_sample_stats.restype = i32
    lib.spechub_draft_sample_stats.argtypes = [ctypes.POINTER(_Desc), vp, vp, vp, vp, vp, vp, vp, vp]
    lib.rrs_draft_sample_stats.restype = i32
    lib.rrs_draft_sample_stats.argtypes = [ctypes.POINTER(_Desc), vp, vp, i32, vp, vp, vp, vp]
    lib.spechub_verify_tree_stats.restype = i32
    lib.spechub_verify_tree_stats.argtypes = [ctypes.POINTER(_Desc), vp, vp, vp, vp, vp,
                                              ctypes.POINTER(_NodeOut), ctypes.POINTER(_SeqOut), vp,
                                              ctypes.c_size_t, vp]
    lib.rrs_verify_tree_stats.restype = i32
    lib.rrs_verify_tree_stats.argtypes = [ctypes.POINTER(_Desc), vp, vp, vp, vp, vp, i32,
                                          ctypes.POINTER(_NodeOut), ctypes.POINTER(_SeqOut), vp,
                                          ctypes.c_size_t, vp]
    lib.spechub_draft_stats_bytes.restype = ctypes.c_size_t
    lib.spechub_draft_stats_bytes.argtypes = [ctypes.POINTER(_Desc)]
    lib.mdsd_compare_draft_sample.restype = i32
    lib.mdsd_compare_draft_sample.argtypes = [ctypes.POINTER(_Desc), vp, vp, ctypes.POINTER(vp), vp, vp,
                                              ctypes.POINTER(vp), vp]
    lib.mdsd_compare_draft_sample_stats.restype = i32
    lib.mdsd_compare_draft_sample_stats.argtypes = [ctypes.POINTER(_Desc), vp, vp, ctypes.POINTER(vp), vp, vp,
                                                    ctypes.POINTER(vp), vp, vp]
    lib.mdsd_compare_verify_tree_stats.restype = i32
    lib.mdsd_compare_verify_tree_stats.argtypes = [ctypes.POINTER(_Desc), vp, vp, vp, ctypes.POINTER(vp), vp,
                                                   ctypes.POINTER(_NodeOut), ctypes.POINTER(_SeqOut), vp,
                                                   ctypes.c_size_t, vp]
    lib.mdsd_compare_verify_tree.restype = i32
    lib.mdsd_compare_verify_tree.argtypes = [ctypes.POINTER(_Desc), vp, vp, ctypes.POINTER(vp), vp,
                                             ctypes.POINTER(_NodeOut), ctypes.POINTER(_SeqOut), vp,
                                             ctypes.c_size_t, vp]
    lib.spechub_verify_tree_static.restype = i32
    lib.spechub_verify_tree_static.argtypes = [ctypes.POINTER(_Desc), vp, vp, vp, vp,
                                               ctypes.POINTER(_NodeOut), ctypes.POINTER(_SeqOut), vp]
    lib.spechub_workspace_bytes.restype = ctypes.c_size_t
    lib.spechub_workspace_bytes.argtypes = [ctypes.POINTER(_Desc)]
    lib.spechub_status_string.restype = ctypes.c_char_p
    lib.spechub_status_string.argtypes = [i32]
    lib.spechub_abi_version.restype = i32
    lib.spechub_abi_version.argtypes = []
    if lib.spechub_abi_version() != ABI_VERSION:
        raise SpecHubError(-101, "library ABI %d != binding ABI %d" % (lib.spechub_abi_version(), ABI_VERSION))
    _lib = lib
    return lib


def abi_version() -> int:
    return int(load_library().spechub_abi_version())


def status_string(code: int) -> str:
    return load_library().spechub_status_string(int(code)).decode()


def _check(code: int):
    if code != 0:
        raise SpecHubError(code, status_string(code))


# tuning hint for the large-vocabulary bf16 kernels: CTAs of a cluster per row (0 = library default)
_split = 0


def set_row_split(ctas: int) -> None:
    """Force 1, 2 or 4 CTAs per row in the large-vocabulary streaming kernels (0 restores the
    default); 8 selects verification with the exponentials resident on chip (SPECHUB_FLAG_RESIDENT)."""
    global _split
    if ctas not in (0, 1, 2, 4, 8):
        raise ValueError("row split must be 0, 1, 2, 4 or 8 (8 = resident)")
    _split = ctas


@dataclass
class Tree:
    """Token tree in level order.  ``child``/``node_kind`` are device tensors or None
    (None = complete binary tree in heap order, every node verifies)."""

    levels: int
    child: Optional[torch.Tensor] = None      # int32 [nodes][k]
    node_kind: Optional[torch.Tensor] = None  # uint8 [nodes]
    k: int = 2                                # drafts (children) per node; > 2 for RRS / RRSw only

    @staticmethod
    def heap(nodes: int, leaves_sample: bool = False, device="cuda") -> "Tree":
        """Complete binary tree of 2^d - 1 nodes.  With ``leaves_sample`` the last level holds
        leaves that only draw the bonus token from p (Figure 2 of the paper)."""
        d = (nodes + 1).bit_length() - 1
        if (1 << d) - 1 != nodes:
            raise ValueError("heap trees have 2^d - 1 nodes")
        kind = None
        if leaves_sample:
            kind = torch.zeros(nodes, dtype=torch.uint8)
            kind[nodes // 2:] = 1
            kind = kind.to(device)
        return Tree(levels=d, child=None, node_kind=kind)

    @staticmethod
    def kary(k: int, levels: int, leaves_sample: bool = False, device="cuda") -> "Tree":
        """Complete k-ary tree with `levels` levels in level order ((k^levels - 1)/(k - 1) nodes)."""
        nodes = (k ** levels - 1) // (k - 1)
        kind = None
        if leaves_sample:
            kind = torch.zeros(nodes, dtype=torch.uint8)
            kind[(k ** (levels - 1) - 1) // (k - 1):] = 1
            kind = kind.to(device)
        return Tree(levels=levels, child=None, node_kind=kind, k=k)

    @staticmethod
    def from_parents(parents, k: int = 2, leaves_sample: bool = True, device="cuda") -> "Tree":
        """Any tree in level order from its parent list (``parents[0] = -1``; every parent index is
        smaller than its child's; at most ``k`` children per node, in the order they are listed):
        unbalanced trees such as the paper's binary Sequoia shapes.  Child slot i of a node is the
        target of its draft i; missing children are -1.  With ``leaves_sample`` the childless
        nodes only draw the bonus token from p."""
        n = len(parents)
        if n < 1 or parents[0] != -1:
            raise ValueError("parents[0] must be -1 (the root)")
        child = [[-1] * k for _ in range(n)]
        depth = [1] * n
        for c in range(1, n):
            p = int(parents[c])
            if not 0 <= p < c:
                raise ValueError("node %d: parent %d must be an earlier node" % (c, p))
            if depth[c - 1] > depth[p] + 1:
                raise ValueError("nodes must be listed level by level")
            slot = next((i for i in range(k) if child[p][i] < 0), None)
            if slot is None:
                raise ValueError("node %d has more than %d children" % (p, k))
            child[p][slot] = c
            depth[c] = depth[p] + 1
        kind = None
        if leaves_sample:
            kind = torch.tensor([1 if all(x < 0 for x in row) else 0 for row in child], dtype=torch.uint8).to(device)
        return Tree(levels=max(depth), child=torch.tensor(child, dtype=torch.int32).to(device), node_kind=kind, k=k)

    def nodes_of_complete_tree(self) -> int:
        return (self.k ** self.levels - 1) // (self.k - 1)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _hold(tensors, stream):
    """Temporaries of a call (a converted temperature vector, a workspace) are freed when the Python
    call returns, while the kernels may still be queued.  On the current stream torch's allocator
    orders the reuse after them; on any other stream it has to be told."""
    if stream is None:
        return
    for t in tensors:
        if t is not None:
            t.record_stream(stream)


def _desc(logits: torch.Tensor, tree: Tree, temperature) -> tuple:
    if logits.dim() != 3 or logits.stride(2) != 1:
        raise ValueError("logits must be [batch][nodes][vocab] with a contiguous vocabulary axis")
    if not logits.is_cuda:
        raise ValueError("logits must live on a CUDA device")
    if logits.dtype == torch.float32:
        dt = F32
    elif logits.dtype == torch.bfloat16:
        dt = BF16
    else:
        raise ValueError("logits must be float32 or bfloat16")
    B, N, V = logits.shape
    d = _Desc()
    d.struct_size = ctypes.sizeof(_Desc)
    d.version = ABI_VERSION
    d.batch, d.nodes, d.vocab, d.k = B, N, V, tree.k
    d.dtype = dt
    d.levels = tree.levels
    d.stride_seq = logits.stride(0) if B > 1 else max(logits.stride(0), (N - 1) * logits.stride(1) + V)
    d.stride_node = logits.stride(1) if N > 1 else max(logits.stride(1), V)
    keep = []
    if isinstance(temperature, torch.Tensor):
        t = temperature.to(device=logits.device, dtype=torch.float32).contiguous()
        if t.shape != (B,):
            raise ValueError("temperature tensor must be [batch]")
        keep.append(t)
        d.temperature = 1.0
        d.temperature_per_seq = t.data_ptr()
    else:
        d.temperature = float(temperature)
        d.temperature_per_seq = None
    if tree.child is not None:
        if tree.child.dtype != torch.int32 or tuple(tree.child.shape) != (N, tree.k) or not tree.child.is_contiguous():
            raise ValueError("child must be a contiguous int32 [nodes][k] tensor")
        d.child = tree.child.data_ptr()
    if tree.node_kind is not None:
        if tree.node_kind.dtype != torch.uint8 or tuple(tree.node_kind.shape) != (N,):
            raise ValueError("node_kind must be a uint8 [nodes] tensor")
        d.node_kind = tree.node_kind.data_ptr()
    d.flags = _split  # SPECHUB_FLAG_SPLIT_n has the value n
    return d, keep


def _same_layout(a: torch.Tensor, b: torch.Tensor):
    if a.shape != b.shape or a.dtype != b.dtype or a.stride() != b.stride() or a.device != b.device:
        raise ValueError("target and draft logits must share shape, dtype, strides and device")


def _check_uniforms(u, B, N, dev, k=2):
    if (u.dtype != torch.float32 or tuple(u.shape) != (B, N, 2 * k + 1) or not u.is_contiguous()
            or u.device != dev):
        raise ValueError("uniforms must be a contiguous float32 [batch][nodes][2k+1] tensor on the logits' device")


def _need_k2(tree):
    if tree.k != 2:
        raise ValueError("SpecHub takes exactly two drafts per node")


def _alloc_stats(lib, d, dev):
    """The caller-owned buffer of per-row draft statistics (16 bytes per row, opaque)."""
    n = lib.spechub_draft_stats_bytes(ctypes.byref(d))
    return torch.empty(max(n, 16) // 4, dtype=torch.int32, device=dev)


def spechub_draft_sample(draft_logits, uniforms, tree: Tree, temperature=1.0, stream=None):
    """Draw the k = 2 SpecHub drafts of every node.  Returns dict(tokens, hub, prob, status)."""
    return _spechub_draft(draft_logits, uniforms, tree, temperature, stream, False)


def spechub_draft_sample_stats(draft_logits, uniforms, tree: Tree, temperature=1.0, stream=None):
    """``spechub_draft_sample`` that also leaves the per-row draft statistics (key ``stats``) for
    ``spechub_verify_tree_stats``."""
    return _spechub_draft(draft_logits, uniforms, tree, temperature, stream, True)


def _spechub_draft(draft_logits, uniforms, tree, temperature, stream, with_stats):
    lib = load_library()
    _need_k2(tree)
    d, keep = _desc(draft_logits, tree, temperature)
    B, N, _ = draft_logits.shape
    dev = draft_logits.device
    _check_uniforms(uniforms, B, N, dev)
    tokens = torch.empty((B, N, 2), dtype=torch.int32, device=dev)
    hub = torch.empty((B, N), dtype=torch.int32, device=dev)
    prob = torch.empty((B, N, 2), dtype=torch.float32, device=dev)
    status = torch.empty((B, N), dtype=torch.int32, device=dev)
    out = dict(tokens=tokens, hub=hub, prob=prob, status=status)
    if with_stats:
        out["stats"] = _alloc_stats(lib, d, dev)
        _check(lib.spechub_draft_sample_stats(ctypes.byref(d), _ptr(draft_logits), _ptr(uniforms), _ptr(tokens),
                                              _ptr(hub), _ptr(prob), _ptr(status), _ptr(out["stats"]),
                                              _stream_ptr(stream)))
    else:
        _check(lib.spechub_draft_sample(ctypes.byref(d), _ptr(draft_logits), _ptr(uniforms), _ptr(tokens),
                                        _ptr(hub), _ptr(prob), _ptr(status), _stream_ptr(stream)))
    _hold(keep + list(out.values()), stream)
    return out


def rrs_draft_sample(draft_logits, uniforms, tree: Tree, without_replacement: bool, temperature=1.0,
                     stream=None):
    """Draw the k = tree.k RRS / RRSw drafts of every node.  Returns dict(tokens, status)."""
    return _rrs_draft(draft_logits, uniforms, tree, without_replacement, temperature, stream, False)


def rrs_draft_sample_stats(draft_logits, uniforms, tree: Tree, without_replacement: bool, temperature=1.0,
                           stream=None):
    """``rrs_draft_sample`` that also leaves the per-row draft statistics (key ``stats``) for
    ``rrs_verify_tree_stats``."""
    return _rrs_draft(draft_logits, uniforms, tree, without_replacement, temperature, stream, True)


def _rrs_draft(draft_logits, uniforms, tree, without_replacement, temperature, stream, with_stats):
    lib = load_library()
    d, keep = _desc(draft_logits, tree, temperature)
    B, N, _ = draft_logits.shape
    dev = draft_logits.device
    _check_uniforms(uniforms, B, N, dev, tree.k)
    tokens = torch.empty((B, N, tree.k), dtype=torch.int32, device=dev)
    status = torch.empty((B, N), dtype=torch.int32, device=dev)
    out = dict(tokens=tokens, status=status)
    if with_stats:
        out["stats"] = _alloc_stats(lib, d, dev)
        _check(lib.rrs_draft_sample_stats(ctypes.byref(d), _ptr(draft_logits), _ptr(uniforms),
                                          int(bool(without_replacement)), _ptr(tokens), _ptr(status),
                                          _ptr(out["stats"]), _stream_ptr(stream)))
    else:
        _check(lib.rrs_draft_sample(ctypes.byref(d), _ptr(draft_logits), _ptr(uniforms),
                                    int(bool(without_replacement)), _ptr(tokens), _ptr(status),
                                    _stream_ptr(stream)))
    _hold(keep + list(out.values()), stream)
    return out


def alloc_verify_outputs(B, N, levels, dev, k=2):
    """Device buffers for one verify call (reusable across calls of the same shape)."""
    return dict(
        accept_idx=torch.empty((B, N), dtype=torch.int32, device=dev),
        token=torch.empty((B, N), dtype=torch.int32, device=dev),
        hub=torch.empty((B, N), dtype=torch.int32, device=dev),
        beta=torch.empty((B, N, k), dtype=torch.float32, device=dev),
        rate=torch.empty((B, N, k + 1), dtype=torch.float32, device=dev),
        status=torch.empty((B, N), dtype=torch.int32, device=dev),
        n_accepted=torch.empty((B,), dtype=torch.int32, device=dev),
        n_emitted=torch.empty((B,), dtype=torch.int32, device=dev),
        path_nodes=torch.empty((B, levels), dtype=torch.int32, device=dev),
        path_tokens=torch.empty((B, levels), dtype=torch.int32, device=dev),
    )


def _verify(method, target_logits, draft_logits, draft_tokens, uniforms, tree, temperature, stream,
            out, probabilities=True, stats=None, with_stats=False):
    lib = load_library()
    _same_layout(target_logits, draft_logits)
    d, keep = _desc(target_logits, tree, temperature)
    B, N, _ = target_logits.shape
    dev = target_logits.device
    if method == "spechub":
        _need_k2(tree)
    _check_uniforms(uniforms, B, N, dev, tree.k)
    if (draft_tokens.dtype != torch.int32 or tuple(draft_tokens.shape) != (B, N, tree.k)
            or not draft_tokens.is_contiguous() or draft_tokens.device != dev):
        raise ValueError("draft_tokens must be a contiguous int32 [batch][nodes][k] tensor")
    if out is None:
        out = alloc_verify_outputs(B, N, tree.levels, dev, tree.k)
    no = _NodeOut(*[out[k].data_ptr() if (probabilities or k not in ("beta", "rate")) else None
                    for k in ("accept_idx", "token", "hub", "beta", "rate", "status")])
    so = _SeqOut(*[out[k].data_ptr() for k in ("n_accepted", "n_emitted", "path_nodes", "path_tokens")])
    ws_bytes = lib.spechub_workspace_bytes(ctypes.byref(d))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev) if ws_bytes else None
    common = (ctypes.byref(d), _ptr(target_logits), _ptr(draft_logits), _ptr(draft_tokens), _ptr(uniforms))
    tail = (ctypes.byref(no), ctypes.byref(so), _ptr(ws), ws_bytes, _stream_ptr(stream))
    if with_stats:
        need = lib.spechub_draft_stats_bytes(ctypes.byref(d))
        if (stats is None or stats.dtype != torch.int32 or not stats.is_contiguous() or stats.device != dev
                or stats.numel() * 4 < need):
            raise ValueError("stats must be the tensor a *_draft_sample_stats call returned for this shape")
        common = common[:3] + (_ptr(stats),) + common[3:]
        if method == "spechub":
            _check(lib.spechub_verify_tree_stats(*common, *tail))
        else:
            _check(lib.rrs_verify_tree_stats(*common, 1 if method == "rrsw" else 0, *tail))
    elif method == "spechub":
        _check(lib.spechub_verify_tree(*common, *tail))
    else:
        _check(lib.rrs_verify_tree(*common, 1 if method == "rrsw" else 0, *tail))
    _hold(keep + [ws, stats] + list(out.values()), stream)
    return out


def spechub_verify_tree(target_logits, draft_logits, draft_tokens, uniforms, tree: Tree,
                        temperature=1.0, stream=None, out=None, probabilities=True):
    """SpecHub verification of every node and the tree walk.  Returns the dict of output
    tensors (see ``alloc_verify_outputs``); pass ``out`` to reuse buffers.  With
    ``probabilities=False`` the library is given no beta / rate buffers (their tensors are left
    untouched) and skips work that only they need."""
    return _verify("spechub", target_logits, draft_logits, draft_tokens, uniforms, tree, temperature,
                   stream, out, probabilities)


def rrs_verify_tree(target_logits, draft_logits, draft_tokens, uniforms, tree: Tree,
                    without_replacement: bool, temperature=1.0, stream=None, out=None, probabilities=True):
    """RRS / RRSw verification of every node and the tree walk."""
    return _verify("rrsw" if without_replacement else "rrs", target_logits, draft_logits, draft_tokens,
                   uniforms, tree, temperature, stream, out, probabilities)


def spechub_verify_tree_stats(target_logits, draft_logits, stats, draft_tokens, uniforms, tree: Tree,
                              temperature=1.0, stream=None, out=None, probabilities=True):
    """``spechub_verify_tree`` given the draft statistics ``spechub_draft_sample_stats`` left for the same
    draft logits, tree and temperature: the first pass reads the target rows only."""
    return _verify("spechub", target_logits, draft_logits, draft_tokens, uniforms, tree, temperature,
                   stream, out, probabilities, stats, True)


def rrs_verify_tree_stats(target_logits, draft_logits, stats, draft_tokens, uniforms, tree: Tree,
                          without_replacement: bool, temperature=1.0, stream=None, out=None,
                          probabilities=True):
    """``rrs_verify_tree`` given the draft statistics ``rrs_draft_sample_stats`` left."""
    return _verify("rrsw" if without_replacement else "rrs", target_logits, draft_logits, draft_tokens,
                   uniforms, tree, temperature, stream, out, probabilities, stats, True)


METHODS = ("spechub", "rrs", "rrsw")


def mdsd_compare_draft_sample(draft_logits, uniforms, tree: Tree, temperature=1.0, stream=None):
    """Draft step of SpecHub, RRS and RRSw on the same q and uniforms.  Returns a dict keyed by
    method name; each entry is what the method's own draft call returns."""
    return _compare_draft(draft_logits, uniforms, tree, temperature, stream, False)


def mdsd_compare_draft_sample_stats(draft_logits, uniforms, tree: Tree, temperature=1.0, stream=None):
    """``mdsd_compare_draft_sample`` that also leaves the per-row draft statistics (key ``stats`` of the
    returned dict, one buffer for the three methods) for ``mdsd_compare_verify_tree_stats``."""
    return _compare_draft(draft_logits, uniforms, tree, temperature, stream, True)


def _compare_draft(draft_logits, uniforms, tree, temperature, stream, with_stats):
    lib = load_library()
    _need_k2(tree)
    d, keep = _desc(draft_logits, tree, temperature)
    B, N, _ = draft_logits.shape
    dev = draft_logits.device
    _check_uniforms(uniforms, B, N, dev)
    tokens = [torch.empty((B, N, 2), dtype=torch.int32, device=dev) for _ in METHODS]
    status = [torch.empty((B, N), dtype=torch.int32, device=dev) for _ in METHODS]
    hub = torch.empty((B, N), dtype=torch.int32, device=dev)
    prob = torch.empty((B, N, 2), dtype=torch.float32, device=dev)
    tp = (ctypes.c_void_p * 3)(*[t.data_ptr() for t in tokens])
    sp = (ctypes.c_void_p * 3)(*[t.data_ptr() for t in status])
    stats = None
    if with_stats:
        stats = _alloc_stats(lib, d, dev)
        _check(lib.mdsd_compare_draft_sample_stats(ctypes.byref(d), _ptr(draft_logits), _ptr(uniforms), tp,
                                                   _ptr(hub), _ptr(prob), sp, _ptr(stats), _stream_ptr(stream)))
    else:
        _check(lib.mdsd_compare_draft_sample(ctypes.byref(d), _ptr(draft_logits), _ptr(uniforms), tp, _ptr(hub),
                                             _ptr(prob), sp, _stream_ptr(stream)))
    _hold(keep + tokens + status + [hub, prob, stats], stream)
    res = dict(spechub=dict(tokens=tokens[0], hub=hub, prob=prob, status=status[0]),
               rrs=dict(tokens=tokens[1], status=status[1]),
               rrsw=dict(tokens=tokens[2], status=status[2]))
    if with_stats:
        res["stats"] = stats
    return res


def mdsd_compare_verify_tree(target_logits, draft_logits, draft_tokens, uniforms, tree: Tree,
                             temperature=1.0, stream=None, out=None, probabilities=True):
    """Verification and tree walk by SpecHub, RRS and RRSw from shared reads of p and q.
    ``draft_tokens`` and ``out`` are dicts keyed by method name (``out`` entries as made by
    ``alloc_verify_outputs``).  Returns ``out``."""
    return _compare_verify(target_logits, draft_logits, draft_tokens, uniforms, tree, temperature, stream, out,
                           probabilities, None, False)


def mdsd_compare_verify_tree_stats(target_logits, draft_logits, stats, draft_tokens, uniforms, tree: Tree,
                                   temperature=1.0, stream=None, out=None, probabilities=True):
    """``mdsd_compare_verify_tree`` given the draft statistics ``mdsd_compare_draft_sample_stats`` left."""
    return _compare_verify(target_logits, draft_logits, draft_tokens, uniforms, tree, temperature, stream, out,
                           probabilities, stats, True)


def _compare_verify(target_logits, draft_logits, draft_tokens, uniforms, tree, temperature, stream, out,
                    probabilities, stats, with_stats):
    lib = load_library()
    _need_k2(tree)
    _same_layout(target_logits, draft_logits)
    d, keep = _desc(target_logits, tree, temperature)
    B, N, _ = target_logits.shape
    dev = target_logits.device
    _check_uniforms(uniforms, B, N, dev)
    for m in METHODS:
        t = draft_tokens[m]
        if t.dtype != torch.int32 or tuple(t.shape) != (B, N, 2) or not t.is_contiguous() or t.device != dev:
            raise ValueError("draft_tokens[%s] must be a contiguous int32 [batch][nodes][2] tensor" % m)
    if out is None:
        out = {m: alloc_verify_outputs(B, N, tree.levels, dev) for m in METHODS}
    no = (_NodeOut * 3)(*[
        _NodeOut(*[out[m][k].data_ptr() if (probabilities or k not in ("beta", "rate")) else None
                   for k in ("accept_idx", "token", "hub", "beta", "rate", "status")]) for m in METHODS])
    so = (_SeqOut * 3)(*[
        _SeqOut(*[out[m][k].data_ptr() for k in ("n_accepted", "n_emitted", "path_nodes", "path_tokens")])
        for m in METHODS])
    tp = (ctypes.c_void_p * 3)(*[draft_tokens[m].data_ptr() for m in METHODS])
    ws_bytes = lib.spechub_workspace_bytes(ctypes.byref(d))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev) if ws_bytes else None
    if with_stats:
        need = lib.spechub_draft_stats_bytes(ctypes.byref(d))
        if (stats is None or stats.dtype != torch.int32 or not stats.is_contiguous() or stats.device != dev
                or stats.numel() * 4 < need):
            raise ValueError("stats must be the tensor a *_draft_sample_stats call returned for this shape")
        _check(lib.mdsd_compare_verify_tree_stats(ctypes.byref(d), _ptr(target_logits), _ptr(draft_logits),
                                                  _ptr(stats), tp, _ptr(uniforms), no, so, _ptr(ws), ws_bytes,
                                                  _stream_ptr(stream)))
    else:
        _check(lib.mdsd_compare_verify_tree(ctypes.byref(d), _ptr(target_logits), _ptr(draft_logits), tp,
                                            _ptr(uniforms), no, so, _ptr(ws), ws_bytes, _stream_ptr(stream)))
    _hold(keep + [ws, stats] + [t for m in METHODS for t in out[m].values()], stream)
    return out


STATIC_MAX_ROWS = 16384


def spechub_verify_tree_static(target_logits, draft_logits, draft_tokens, uniforms, tree: Tree,
                               temperature=1.0, stream=None, out=None):
    """SpecHub verification and tree walk through the entry point that allocates nothing on the
    device: for callers whose GPU memory is spoken for (a server's pre-reserved pools, another
    framework's memory plan) or who may not enter the allocator at all.  The library keeps its
    intermediate per-row records in a static array of its own, so at most ``STATIC_MAX_ROWS``
    (batch x nodes) rows per call, and calls on one device must not overlap.  Pass ``out`` (from
    ``alloc_verify_outputs``) to keep this wrapper from allocating the result tensors too."""
    lib = load_library()
    _need_k2(tree)
    _same_layout(target_logits, draft_logits)
    d, keep = _desc(target_logits, tree, temperature)
    B, N, _ = target_logits.shape
    dev = target_logits.device
    _check_uniforms(uniforms, B, N, dev)
    if (draft_tokens.dtype != torch.int32 or tuple(draft_tokens.shape) != (B, N, 2)
            or not draft_tokens.is_contiguous() or draft_tokens.device != dev):
        raise ValueError("draft_tokens must be a contiguous int32 [batch][nodes][2] tensor")
    if out is None:
        out = alloc_verify_outputs(B, N, tree.levels, dev)
    no = _NodeOut(*[out[k].data_ptr() for k in ("accept_idx", "token", "hub", "beta", "rate", "status")])
    so = _SeqOut(*[out[k].data_ptr() for k in ("n_accepted", "n_emitted", "path_nodes", "path_tokens")])
    _check(lib.spechub_verify_tree_static(ctypes.byref(d), _ptr(target_logits), _ptr(draft_logits),
                                          _ptr(draft_tokens), _ptr(uniforms), ctypes.byref(no),
                                          ctypes.byref(so), _stream_ptr(stream)))
    _hold(keep + list(out.values()), stream)
    return out


def workspace_bytes(logits, tree: Tree, temperature=1.0) -> int:
    d, _ = _desc(logits, tree, temperature)
    return int(load_library().spechub_workspace_bytes(ctypes.byref(d)))
