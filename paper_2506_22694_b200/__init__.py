"""B200-native VocabTrim hot path: thin Python binding over the C-ABI CUDA library.

Everything here is argument marshalling.  Tensors are torch CUDA tensors used only as device
memory; every step of the path (histogram, top-K selection, head gather, trimmed head with its
sampling epilogue and the remap) runs in the hand-written sm_100a kernels of libvocabtrim.so.
There is no CPU or PyTorch fallback: if the library is missing or a call fails, an exception is
raised.

Names follow the C header (include/vocabtrim.h): vt_histogram, vt_select_topk, vt_build_vocab,
vt_trim_head, vt_draft_head, ...  `map` is in rank order (map[0] = most frequent id).
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_char_p, c_double, c_float, c_int, c_int32, c_int64, c_size_t, c_uint32, c_uint64, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libvocabtrim.so")

VT_OK = 0
VT_OP_HISTOGRAM, VT_OP_SELECT_TOPK, VT_OP_BUILD_VOCAB, VT_OP_TRIM_HEAD = 0, 1, 2, 3
VT_OP_DRAFT_HEAD, VT_OP_DRAFT_HEAD_HOST, VT_OP_BUILD_VOCAB_HOST = 4, 5, 6
VT_FLAG_BAD_ID, VT_FLAG_BAD_MAP, VT_FLAG_BAD_TEMP, VT_FLAG_NAN_ROW, VT_FLAG_TIMEOUT = 1, 2, 4, 8, 16
VT_MAX_TOPK = 64
VT_CTRL_BYTES = 256

EXPORTS = (
    "vt_workspace_bytes", "vt_workspace_init", "vt_workspace_set_wait_limit", "vt_read_status", "vt_status_str", "vt_launch_count",
    "vt_last_cuda_error",
    "vt_histogram", "vt_histogram_folded", "vt_select_topk", "vt_build_vocab", "vt_build_vocab_host", "vt_trim_head",
    "vt_draft_head", "vt_draft_head_debug", "vt_draft_head_host", "vt_select_topk_static",
    "vt_draft_head_overlapped", "vt_select_topp", "vt_select_minfreq", "vt_verify_greedy", "vt_mbsu", "vt_tree_expand", "vt_tree_rerank", "vt_draft_head_expand",
)


class VocabTrimError(RuntimeError):
    def __init__(self, call: str, status: int):
        self.status = status
        detail = " [%s]" % lib().vt_last_cuda_error().decode() if status == 4 else ""
        super().__init__("%s failed: %s (status %d)%s" % (call, status_str(status), status, detail))


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libvocabtrim.so; raises if it has not been built (python -m paper_2506_22694_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libvocabtrim.so is missing: build it with "
                               "`python -m paper_2506_22694_b200.build` (no fallback path exists)")
        L = ctypes.CDLL(LIB_PATH)
        L.vt_workspace_bytes.restype = c_size_t
        L.vt_workspace_bytes.argtypes = [c_int, c_int64, c_int32, c_int32, c_int32, c_int32, c_int32]
        L.vt_workspace_init.argtypes = [c_void_p, c_size_t, c_void_p]
        L.vt_read_status.argtypes = [c_void_p, c_void_p, ctypes.POINTER(c_uint32), ctypes.POINTER(c_uint64)]
        L.vt_workspace_set_wait_limit.argtypes = [c_void_p, c_uint64, c_void_p]
        L.vt_status_str.restype = c_char_p
        L.vt_status_str.argtypes = [c_int]
        L.vt_launch_count.restype = c_uint64
        L.vt_last_cuda_error.restype = c_char_p
        L.vt_histogram.argtypes = [c_void_p, c_int64, c_int32, c_void_p, c_int, c_void_p, c_size_t, c_void_p]
        L.vt_histogram_folded.argtypes = [c_void_p, c_int64, c_int32, c_int32, c_void_p, c_void_p]
        L.vt_select_topk.argtypes = [c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
        L.vt_select_topk_static.argtypes = [c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p]
        L.vt_select_topp.argtypes = [c_void_p, c_int32, c_double, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
        L.vt_select_minfreq.argtypes = [c_void_p, c_int32, c_uint32, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
        L.vt_verify_greedy.argtypes = [c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
        L.vt_mbsu.argtypes = [c_double, c_double, c_double, c_int32]
        L.vt_mbsu.restype = c_double
        L.vt_tree_expand.argtypes = [c_void_p, c_void_p, c_int32, c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p]
        L.vt_draft_head_expand.argtypes = [c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p, c_size_t, c_void_p]
        L.vt_tree_rerank.argtypes = [c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p]
        L.vt_build_vocab.argtypes = [c_void_p, c_int64, c_int32, c_int32, c_void_p, c_void_p, c_void_p,
                                     c_size_t, c_void_p]
        L.vt_build_vocab_host.argtypes = L.vt_build_vocab.argtypes
        L.vt_trim_head.argtypes = [c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p]
        head = [c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p, c_int32, c_void_p,
                c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
        L.vt_draft_head.argtypes = head
        L.vt_draft_head_overlapped.argtypes = head
        L.vt_draft_head_host.argtypes = head
        L.vt_draft_head_debug.argtypes = head + [c_void_p, c_void_p]
        _lib = L
    return _lib


def status_str(status: int) -> str:
    return lib().vt_status_str(int(status)).decode()


def launch_count() -> int:
    return int(lib().vt_launch_count())


def _check(call: str, status: int) -> None:
    if status != VT_OK:
        raise VocabTrimError(call, status)


def _ptr(t):
    return c_void_p(t.data_ptr()) if t is not None else c_void_p(0)


def _stream() -> c_void_p:
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError("%s must be a contiguous CUDA tensor of dtype %s" % (name, dtype))
    return t


def workspace_bytes(op: int, n: int = 0, V: int = 0, K: int = 0, d: int = 0, B: int = 0, topk: int = 0) -> int:
    return int(lib().vt_workspace_bytes(op, n, V, K, d, B, topk))


class Workspace:
    """Caller-owned scratch for the library: a 256-byte-aligned device buffer whose control block
    has been cleared once (vt_workspace_init).  One workspace serves one stream at a time."""

    def __init__(self, nbytes: int, device="cuda"):
        if nbytes <= 0:
            raise ValueError("unsupported shape: the library reported a zero-size workspace")
        self.nbytes = int(nbytes)
        self.buf = torch.empty(self.nbytes + 256, dtype=torch.uint8, device=device)
        off = (-self.buf.data_ptr()) % 256
        self.ptr = self.buf.data_ptr() + off
        _check("vt_workspace_init", lib().vt_workspace_init(c_void_p(self.ptr), self.nbytes, _stream()))

    def set_wait_limit(self, nanoseconds: int) -> None:
        """Bound of every device-side wait of the streaming head kernel (0 = the default of 2 s)."""
        _check("vt_workspace_set_wait_limit",
               lib().vt_workspace_set_wait_limit(c_void_p(self.ptr), int(nanoseconds), _stream()))

    def read_status(self):
        """Synchronises the current stream; returns (status, flags, n_bad) and clears the flags."""
        flags, bad = c_uint32(0), c_uint64(0)
        st = lib().vt_read_status(c_void_p(self.ptr), _stream(), ctypes.byref(flags), ctypes.byref(bad))
        return int(st), int(flags.value), int(bad.value)


def _ws(ws: Workspace | None, need: int, like: torch.Tensor) -> Workspace:
    if ws is None:
        return Workspace(need, like.device)
    if ws.nbytes < need:
        raise VocabTrimError("workspace too small (%d < %d)" % (ws.nbytes, need), 3)
    return ws


def vt_histogram(ids: torch.Tensor, V: int, counts: torch.Tensor | None = None, accumulate: bool = False,
                 ws: Workspace | None = None) -> torch.Tensor:
    """Algorithm 1.  ids int32 [n] -> counts int32 storage holding uint32 values [V]."""
    _dev(ids, torch.int32, "ids")
    if counts is None:
        counts = torch.empty(V, dtype=torch.int32, device=ids.device)
        accumulate = False
    _dev(counts, torch.int32, "counts")
    ws = _ws(ws, workspace_bytes(VT_OP_HISTOGRAM, ids.numel(), V), ids)
    _check("vt_histogram", lib().vt_histogram(_ptr(ids), ids.numel(), V, _ptr(counts), int(bool(accumulate)),
                                              c_void_p(ws.ptr), ws.nbytes, _stream()))
    return counts


def vt_histogram_folded(ids: torch.Tensor, V: int, bins: int, counts: torch.Tensor | None = None) -> torch.Tensor:
    """Measurement aid: counts[id mod bins] over the ids inside [0,V), all bins directly indexed in
    shared memory (bins <= 57344)."""
    _dev(ids, torch.int32, "ids")
    if counts is None:
        counts = torch.empty(bins, dtype=torch.int32, device=ids.device)
    _dev(counts, torch.int32, "counts")
    _check("vt_histogram_folded", lib().vt_histogram_folded(_ptr(ids), ids.numel(), V, bins, _ptr(counts), _stream()))
    return counts


def vt_select_topk(counts: torch.Tensor, K: int, ws: Workspace | None = None):
    """Eq. 1 (token selection).  counts [V] -> (map int32 [K], inv_map int32 [V])."""
    _dev(counts, torch.int32, "counts")
    V = counts.numel()
    map_ = torch.empty(K, dtype=torch.int32, device=counts.device)
    inv = torch.empty(V, dtype=torch.int32, device=counts.device)
    ws = _ws(ws, workspace_bytes(VT_OP_SELECT_TOPK, 0, V, K), counts)
    _check("vt_select_topk", lib().vt_select_topk(_ptr(counts), V, K, _ptr(map_), _ptr(inv), c_void_p(ws.ptr),
                                                  ws.nbytes, _stream()))
    return map_, inv


def _select_cut(counts: torch.Tensor, ws, call, *arg):
    _dev(counts, torch.int32, "counts")
    V = counts.numel()
    map_ = torch.empty(V, dtype=torch.int32, device=counts.device)
    inv = torch.empty(V, dtype=torch.int32, device=counts.device)
    k_out = torch.empty(1, dtype=torch.int32, device=counts.device)
    ws = _ws(ws, workspace_bytes(VT_OP_SELECT_TOPK, 0, V, V), counts)
    fn = getattr(lib(), call)
    _check(call, fn(_ptr(counts), V, *arg, _ptr(map_), _ptr(inv), _ptr(k_out), c_void_p(ws.ptr), ws.nbytes, _stream()))
    return k_out, map_, inv


def vt_select_topp(counts: torch.Tensor, p: float, ws: Workspace | None = None):
    """Top-P selection (Method section): returns (K device int32 [1], map [V] whose first K entries are the trimmed vocabulary, inv_map [V])."""
    return _select_cut(counts, ws, "vt_select_topp", c_double(float(p)))


def vt_select_minfreq(counts: torch.Tensor, min_count: int, ws: Workspace | None = None):
    """Minimum-frequency selection (Method section): returns (K device int32 [1], map [V] (first K entries), inv_map [V])."""
    return _select_cut(counts, ws, "vt_select_minfreq", c_uint32(int(min_count)))


def tree_pool(capacity: int, device="cuda"):
    """Caller-owned node pool of vt_tree_expand / vt_tree_rerank: (token, parent, score) tensors."""
    return (torch.empty(capacity, dtype=torch.int32, device=device),
            torch.empty(capacity, dtype=torch.int32, device=device),
            torch.empty(capacity, dtype=torch.float32, device=device))


def vt_tree_expand(cand_ids: torch.Tensor, cand_logprobs: torch.Tensor, frontier_nodes: torch.Tensor | None,
                   pool, pool_base: int, n_front: int, col0: int = 0) -> torch.Tensor:
    """One depth of the draft-tree expansion (Settings).  cand_* are [B, col0+topk] device tensors (the
    head's outputs with col0=1); returns the next frontier's pool indices [n_front], best first."""
    _dev(cand_ids, torch.int32, "cand_ids")
    _dev(cand_logprobs, torch.float32, "cand_logprobs")
    B, ld = cand_ids.shape
    if tuple(cand_logprobs.shape) != (B, ld):
        raise ValueError("cand_ids and cand_logprobs must have the same shape")
    tok, par, sc = pool
    _dev(tok, torch.int32, "pool token"), _dev(par, torch.int32, "pool parent"), _dev(sc, torch.float32, "pool score")
    if frontier_nodes is not None and _dev(frontier_nodes, torch.int32, "frontier_nodes").numel() != B:
        raise ValueError("frontier_nodes must have B entries")
    nxt = torch.empty(n_front, dtype=torch.int32, device=cand_ids.device)
    _check("vt_tree_expand", lib().vt_tree_expand(
        _ptr(cand_ids), _ptr(cand_logprobs), B, ld - col0, ld, col0, _ptr(frontier_nodes), _ptr(tok), _ptr(par),
        _ptr(sc), pool_base, min(tok.numel(), par.numel(), sc.numel()), n_front, _ptr(nxt), _stream()))
    return nxt


def vt_draft_head_expand(h: torch.Tensor, W_trim: torch.Tensor, map_: torch.Tensor | None, temp: torch.Tensor,
                         topk: int, uniforms: torch.Tensor | None, frontier_nodes: torch.Tensor | None, pool,
                         pool_base: int, n_front: int, ws: Workspace | None = None, out=None):
    """One tree depth in one call: the head (as vt_draft_head(..., overlapped=True)) and the expansion of
    its candidates into the node pool.  Returns (out_ids, out_logprobs, next_frontier [n_front])."""
    _dev(h, torch.bfloat16, "h")
    _dev(W_trim, torch.bfloat16, "W_trim")
    _dev(temp, torch.float32, "temp")
    B, d = h.shape
    K = W_trim.shape[0]
    if W_trim.shape[1] != d or temp.numel() != B:
        raise ValueError("shape mismatch between h, W_trim and temp")
    if map_ is not None and _dev(map_, torch.int32, "map").numel() != K:
        raise ValueError("map must have K entries")
    if uniforms is not None and tuple(_dev(uniforms, torch.float32, "uniforms").shape) != (B, K):
        raise ValueError("uniforms must be [B,K]")
    if frontier_nodes is not None and _dev(frontier_nodes, torch.int32, "frontier_nodes").numel() != B:
        raise ValueError("frontier_nodes must have B entries")
    tok, par, sc = pool
    _dev(tok, torch.int32, "pool token"), _dev(par, torch.int32, "pool parent"), _dev(sc, torch.float32, "pool score")
    if out is None:
        out = (torch.empty((B, 1 + topk), dtype=torch.int32, device=h.device),
               torch.empty((B, 1 + topk), dtype=torch.float32, device=h.device))
    ids, lps = out
    nxt = torch.empty(n_front, dtype=torch.int32, device=h.device)
    ws = _ws(ws, workspace_bytes(VT_OP_DRAFT_HEAD, 0, 0, K, d, B, topk), h)
    _check("vt_draft_head_expand", lib().vt_draft_head_expand(
        _ptr(h), _ptr(W_trim), _ptr(map_), B, K, d, _ptr(temp), topk, _ptr(uniforms), _ptr(ids), _ptr(lps),
        _ptr(frontier_nodes), _ptr(tok), _ptr(par), _ptr(sc), pool_base, min(tok.numel(), par.numel(), sc.numel()),
        n_front, _ptr(nxt), c_void_p(ws.ptr), ws.nbytes, _stream()))
    return ids, lps, nxt


def vt_tree_rerank(pool, n: int, budget: int):
    """Final draft of the tree (Settings): returns (nodes, token, parent), each int32 [budget]."""
    tok, par, sc = pool
    _dev(tok, torch.int32, "pool token"), _dev(par, torch.int32, "pool parent"), _dev(sc, torch.float32, "pool score")
    if n > min(tok.numel(), par.numel(), sc.numel()):
        raise ValueError("n exceeds the pool")
    outs = [torch.empty(budget, dtype=torch.int32, device=tok.device) for _ in range(3)]
    _check("vt_tree_rerank", lib().vt_tree_rerank(_ptr(tok), _ptr(par), _ptr(sc), n, budget, _ptr(outs[0]),
                                                  _ptr(outs[1]), _ptr(outs[2]), _stream()))
    return tuple(outs)


def vt_verify_greedy(token: torch.Tensor, parent: torch.Tensor | None, target: torch.Tensor,
                     tokens_total: torch.Tensor | None = None):
    """Greedy verification (Experiments section; Algorithm 2's accept loop) of S blocks.

    token [S,N], parent [S,N] or None (chains), target [S,N+1], all int32 on the device.  Returns
    (n_accept [S], path [S,N], emitted [S,N+1]); `tokens_total` (int64 [1], device) is added to."""
    _dev(token, torch.int32, "token")
    _dev(target, torch.int32, "target")
    S, N = token.shape
    if tuple(target.shape) != (S, N + 1):
        raise ValueError("target must be [S, N+1]")
    if parent is not None:
        _dev(parent, torch.int32, "parent")
        if tuple(parent.shape) != (S, N):
            raise ValueError("parent must be [S, N]")
    if tokens_total is not None:
        _dev(tokens_total, torch.int64, "tokens_total")
    n_accept = torch.empty(S, dtype=torch.int32, device=token.device)
    path = torch.empty(S, N, dtype=torch.int32, device=token.device)
    emitted = torch.empty(S, N + 1, dtype=torch.int32, device=token.device)
    _check("vt_verify_greedy", lib().vt_verify_greedy(
        _ptr(token), _ptr(parent) if parent is not None else None, _ptr(target), S, N, _ptr(n_accept),
        _ptr(path), _ptr(emitted), _ptr(tokens_total) if tokens_total is not None else None, _stream()))
    return n_accept, path, emitted


def vt_mbsu(tau: float, draft_params: float, target_params: float, gamma: int) -> float:
    """Memory-bound speed-up tau / (c*gamma + 1), c = draft_params / target_params (host arithmetic)."""
    return float(lib().vt_mbsu(float(tau), float(draft_params), float(target_params), int(gamma)))


def vt_select_topk_static(counts: torch.Tensor, K: int, out=None):
    """vt_select_topk for callers that may not allocate: the scratch is a fixed array inside the
    library (vocabularies up to VT_STATIC_SELECT_MAX_V ids).  Pass `out` = (map [K], inv_map [V])
    to keep this wrapper allocation-free as well; calls on different streams must not overlap."""
    _dev(counts, torch.int32, "counts")
    V = counts.numel()
    if out is None:
        out = (torch.empty(K, dtype=torch.int32, device=counts.device),
               torch.empty(V, dtype=torch.int32, device=counts.device))
    map_, inv = out
    _check("vt_select_topk_static", lib().vt_select_topk_static(_ptr(counts), V, K, _ptr(map_), _ptr(inv), _stream()))
    return map_, inv


def vt_build_vocab(ids: torch.Tensor, V: int, K: int, ws: Workspace | None = None):
    """Algorithm 1 + Eq. 1 (token selection).  Device ids -> (map [K], inv_map [V]).  A CPU (ideally pinned)
    ids tensor goes through vt_build_vocab_host, which streams it to the device in chunks."""
    if not ids.is_cuda:
        return vt_build_vocab_host(ids, V, K, ws)
    _dev(ids, torch.int32, "ids")
    map_ = torch.empty(K, dtype=torch.int32, device=ids.device)
    inv = torch.empty(V, dtype=torch.int32, device=ids.device)
    ws = _ws(ws, workspace_bytes(VT_OP_BUILD_VOCAB, ids.numel(), V, K), ids)
    _check("vt_build_vocab", lib().vt_build_vocab(_ptr(ids), ids.numel(), V, K, _ptr(map_), _ptr(inv),
                                                  c_void_p(ws.ptr), ws.nbytes, _stream()))
    return map_, inv


def vt_build_vocab_host(ids_host: torch.Tensor, V: int, K: int, ws: Workspace | None = None, device="cuda",
                        out=None):
    if ids_host.is_cuda or ids_host.dtype != torch.int32 or not ids_host.is_contiguous():
        raise TypeError("ids_host must be a contiguous CPU int32 tensor")
    if out is None:
        out = (torch.empty(K, dtype=torch.int32, device=device), torch.empty(V, dtype=torch.int32, device=device))
    map_, inv = out
    ws = _ws(ws, workspace_bytes(VT_OP_BUILD_VOCAB_HOST, ids_host.numel(), V, K), map_)
    _check("vt_build_vocab_host", lib().vt_build_vocab_host(
        c_void_p(ids_host.data_ptr()), ids_host.numel(), V, K, _ptr(map_), _ptr(inv), c_void_p(ws.ptr),
        ws.nbytes, _stream()))
    return map_, inv


def vt_trim_head(W_full: torch.Tensor, map_: torch.Tensor, W_trim: torch.Tensor | None = None,
                 ws: Workspace | None = None) -> torch.Tensor:
    """Eq. 1 (head restriction).  W_full bf16 [V,d], map int32 [K] -> W_trim bf16 [K,d]."""
    _dev(W_full, torch.bfloat16, "W_full")
    _dev(map_, torch.int32, "map")
    V, d = W_full.shape
    K = map_.numel()
    if W_trim is None:
        W_trim = torch.empty((K, d), dtype=torch.bfloat16, device=W_full.device)
    _dev(W_trim, torch.bfloat16, "W_trim")
    _check("vt_trim_head", lib().vt_trim_head(_ptr(W_full), _ptr(map_), _ptr(W_trim), V, K, d,
                                              c_void_p(ws.ptr if ws else 0), _stream()))
    return W_trim


def vt_draft_head(h: torch.Tensor, W_trim: torch.Tensor, map_: torch.Tensor | None, temp: torch.Tensor,
                  topk: int, uniforms: torch.Tensor | None = None, ws: Workspace | None = None,
                  out=None, debug: bool = False, overlapped: bool = False):
    """Algorithm 2 (the drafter's head over the trimmed vocabulary and the index mapping; head part).  Returns (out_ids int32 [B,1+topk], out_logprobs fp32
    [B,1+topk]); with debug=True also (logits fp32 [B,K], lse fp32 [B]).  overlapped=True uses
    vt_draft_head_overlapped (drafting loops with static weights; see the header)."""
    _dev(h, torch.bfloat16, "h")
    _dev(W_trim, torch.bfloat16, "W_trim")
    _dev(temp, torch.float32, "temp")
    B, d = h.shape
    K = W_trim.shape[0]
    if W_trim.shape[1] != d or temp.numel() != B:
        raise ValueError("shape mismatch between h, W_trim and temp")
    if map_ is not None and _dev(map_, torch.int32, "map").numel() != K:
        raise ValueError("map must have K entries")
    if uniforms is not None and tuple(_dev(uniforms, torch.float32, "uniforms").shape) != (B, K):
        raise ValueError("uniforms must be [B,K]")
    if out is None:
        out = (torch.empty((B, 1 + topk), dtype=torch.int32, device=h.device),
               torch.empty((B, 1 + topk), dtype=torch.float32, device=h.device))
    ids, lps = out
    ws = _ws(ws, workspace_bytes(VT_OP_DRAFT_HEAD, 0, 0, K, d, B, topk), h)
    args = [_ptr(h), _ptr(W_trim), _ptr(map_), B, K, d, _ptr(temp), topk, _ptr(uniforms), _ptr(ids), _ptr(lps),
            c_void_p(ws.ptr), ws.nbytes, _stream()]
    if debug:
        logits = torch.empty((B, K), dtype=torch.float32, device=h.device)
        lse = torch.empty(B, dtype=torch.float32, device=h.device)
        _check("vt_draft_head_debug", lib().vt_draft_head_debug(*args, _ptr(logits), _ptr(lse)))
        return ids, lps, logits, lse
    if overlapped:
        _check("vt_draft_head_overlapped", lib().vt_draft_head_overlapped(*args))
    else:
        _check("vt_draft_head", lib().vt_draft_head(*args))
    return ids, lps


def vt_draft_head_host(h_host: torch.Tensor, W_trim: torch.Tensor, map_: torch.Tensor | None,
                       temp_host: torch.Tensor, topk: int, uniforms_host: torch.Tensor | None,
                       ws: Workspace, out_host):
    """vt_draft_head with the per-step tensors in (pinned) host memory; W_trim and map stay on the
    device.  Enqueues copies and kernels on the current stream and returns; synchronise before
    reading out_host = (ids int32 [B,1+topk], logprobs fp32 [B,1+topk]) CPU tensors."""
    B, d = h_host.shape
    K = W_trim.shape[0]
    ids, lps = out_host
    _check("vt_draft_head_host", lib().vt_draft_head_host(
        c_void_p(h_host.data_ptr()), _ptr(W_trim), _ptr(map_), B, K, d, c_void_p(temp_host.data_ptr()), topk,
        c_void_p(uniforms_host.data_ptr() if uniforms_host is not None else 0), c_void_p(ids.data_ptr()),
        c_void_p(lps.data_ptr()), c_void_p(ws.ptr), ws.nbytes, _stream()))
    return ids, lps
