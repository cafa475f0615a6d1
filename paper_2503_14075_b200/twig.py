"""ctypes binding of libtwig.so: the same entry points as include/twig.h.

Argument marshalling only.  Tensors are torch CUDA tensors (torch supplies the
device memory and the stream); every step of the path runs in the library's
kernels.  There is no fallback: if the library is missing this module raises
at import, and a non-zero status raises ``TwigError``.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

_LIB_PATH = _build.LIB
if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build it with `python -m paper_2503_14075_b200.build` "
        "(nvcc, sm_100a); there is no CPU fallback")
_lib = C.CDLL(_LIB_PATH)

STATUS_NAMES = {0: "TWIG_OK", 1: "TWIG_ERR_NULL", 2: "TWIG_ERR_SHAPE", 3: "TWIG_ERR_UNSUPPORTED",
                4: "TWIG_ERR_WORKSPACE", 5: "TWIG_ERR_CUDA", 6: "TWIG_ERR_ALIGN"}
DEV_OK, DEV_BAD_LAYOUT, DEV_BAD_KEEP, DEV_BAD_INDEX, DEV_BAD_TREE, DEV_OVERFLOW, DEV_INTERNAL = range(7)
MAX_NODES, MAX_VISUAL, MAX_BATCH = 64, 16384, 4096

EXPORTS = ["twig_status_str", "twig_set_launch_overlap", "twig_workspace_bytes", "tree_attention_workspace_bytes", "tree_verify_attention_ex", "ttp_score", "ttp_score_gated", "ttp_multiquery_workspace_bytes", "ttp_score_multiquery", "ttp_score_noalloc", "ttp_topk", "ttp_compact", "ttp_compact_rows",
           "ttp_score_topk_compact", "tree_verify_attention", "tree_reset", "tree_expand_level", "tree_select_expansion", "tree_finalize", "tree_grow_level", "tree_base_argmax", "tree_accept_compact", "chain_draft_reset", "chain_draft_step"]


class TwigError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__(f"{STATUS_NAMES.get(code, code)}: {_lib.twig_status_str(code).decode()}")


class KV(C.Structure):
    """Mirror of ``twig_kv`` (strides in elements)."""
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p),
                ("stride_layer", C.c_int64), ("stride_batch", C.c_int64),
                ("stride_head", C.c_int64), ("stride_pos", C.c_int64),
                ("n_layers", C.c_int32), ("batch", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("max_len", C.c_int32)]

    @classmethod
    def of(cls, k: torch.Tensor, v: torch.Tensor) -> "KV":
        """k, v: [n_layers, batch, n_kv_heads, max_len, head_dim] bf16 CUDA tensors."""
        assert k.dim() == 5 and k.shape == v.shape and k.stride() == v.stride() and k.stride(4) == 1
        kv = cls(k.data_ptr(), v.data_ptr(), k.stride(0), k.stride(1), k.stride(2), k.stride(3),
                 k.shape[0], k.shape[1], k.shape[2], k.shape[4], k.shape[3])
        kv._keep = (k, v)
        return kv


_vp, _i32, _i64, _f32, _sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t
_kvp = C.POINTER(KV)
_lib.twig_status_str.restype = C.c_char_p
_lib.twig_status_str.argtypes = [C.c_int]
_lib.twig_set_launch_overlap.restype = C.c_int32
_lib.twig_set_launch_overlap.argtypes = [C.c_int32]
_lib.tree_attention_workspace_bytes.restype = _sz
_lib.tree_attention_workspace_bytes.argtypes = [_i32] * 3
_lib.twig_workspace_bytes.restype = _sz
_lib.twig_workspace_bytes.argtypes = [_i32] * 5
_lib.ttp_score.restype = C.c_int
_lib.ttp_score.argtypes = [_vp, _vp, _i64, _i64, _i64, _i32, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _i32,
                           _f32, _vp, _i32, _vp, _vp, _sz, _vp]
_lib.ttp_score_gated.restype = C.c_int
_lib.ttp_score_gated.argtypes = [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _i32, _vp, _vp, _vp, _i32, _i32, _i32, _i32,
                                 _i32, _f32, _vp, _i32, _vp, _vp, _sz, _vp]
_lib.ttp_multiquery_workspace_bytes.restype = _sz
_lib.ttp_multiquery_workspace_bytes.argtypes = [_i32] * 5
_lib.ttp_score_multiquery.restype = C.c_int
_lib.ttp_score_multiquery.argtypes = [_vp, _i32, _vp, _i64, _i64, _i64, _i32, _vp, _vp, _vp, _i32, _i32, _i32, _i32,
                                      _f32, _vp, _i32, _vp, _vp, _sz, _vp]
_lib.ttp_score_noalloc.restype = C.c_int
_lib.ttp_score_noalloc.argtypes = [_vp, _vp, _i64, _i64, _i64, _i32, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _i32,
                                   _f32, _vp, _i32, _vp, _vp]
NOALLOC_SCRATCH_BYTES = 4 << 20
_lib.ttp_topk.restype = C.c_int
_lib.ttp_topk.argtypes = [_vp, _vp, _vp, _i32, _i32, _i32, _vp, _vp, _vp]
_lib.ttp_compact.restype = C.c_int
_lib.ttp_compact.argtypes = [_kvp, _kvp, _vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp]
_lib.ttp_compact_rows.restype = C.c_int
_lib.ttp_compact_rows.argtypes = [_vp, _vp, _i64, _i64, _i64, _i32, _i64, _i64, _i32, _i32, _vp, _i32, _vp, _vp, _vp,
                                  _vp, _vp, _vp, _vp]
_lib.ttp_score_topk_compact.restype = C.c_int
_lib.ttp_score_topk_compact.argtypes = [_vp, _vp, _i64, _i64, _i64, _i32, _vp, _vp, _vp, _vp, _i32, _i32,
                                        _f32, _vp, _i32, _vp, _i32, _kvp, _kvp, _vp, _vp, _i32, _vp, _vp,
                                        _vp, _sz, _vp]
_lib.tree_verify_attention.restype = C.c_int
_lib.tree_verify_attention.argtypes = [_vp, _vp, _vp, _kvp, _i32, _vp, _vp, _vp, _i32, _i32, _f32, _vp, _vp,
                                       _vp, _vp, _sz, _vp]
_lib.tree_verify_attention_ex.restype = C.c_int
_lib.tree_verify_attention_ex.argtypes = _lib.tree_verify_attention.argtypes + [C.c_uint32]
# per-call flags of tree_verify_attention_ex
ATTN_EARLY_PREFIX, ATTN_PLAIN_LAUNCH, ATTN_EARLY_QUERY = 1, 1 << 4, 1 << 5
ATTN_KERNEL_AUTO, ATTN_KERNEL_MMA, ATTN_KERNEL_TCGEN05, ATTN_KERNEL_STREAM = 0, 1, 2, 3


def attn_flags(kernel=ATTN_KERNEL_AUTO, early_prefix=False, splits=0, plain_launch=False, stream_policy=0,
               early_query=False) -> int:
    """Packs the flags word of tree_verify_attention_ex (stream_policy: 0 the kernel's choice,
    1 equal shares of the key tiles, 2 whole items)."""
    return (int(kernel) << 1) | (ATTN_EARLY_PREFIX if early_prefix else 0) | (int(splits) << 8) | \
        (ATTN_PLAIN_LAUNCH if plain_launch else 0) | (int(stream_policy) << 12) | \
        (ATTN_EARLY_QUERY if early_query else 0)


_lib.tree_reset.restype = C.c_int
_lib.tree_reset.argtypes = [_vp, _vp, _vp, _i32, _i32, _vp]
_lib.tree_expand_level.restype = C.c_int
_lib.tree_expand_level.argtypes = [_vp, _i32, _i64, _i32, _i32, _vp, _i32, _i32, _vp, _vp, _vp, _i32, _i32, _vp, _vp]
_lib.tree_select_expansion.restype = C.c_int
_lib.tree_select_expansion.argtypes = [_vp, _i32, _i32, _i32, _i32, _vp, _i32, _vp, _vp]
_lib.tree_finalize.restype = C.c_int
_lib.tree_finalize.argtypes = [_vp, _vp, _vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _i32, _i32, _vp, _vp]
_lib.tree_grow_level.restype = C.c_int
_lib.tree_grow_level.argtypes = [_vp, _i32, _i64, _i32, _i32, _vp, _i32, _i32, _vp, _vp, _vp, _i32, _i32,
                                 _i32, _vp, _i32, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp]
_lib.tree_base_argmax.restype = C.c_int
_lib.tree_base_argmax.argtypes = [_vp, _i32, _i64, _i32, _vp, _i32, _i32, _vp, _vp, _vp]
_lib.chain_draft_reset.restype = C.c_int
_lib.chain_draft_reset.argtypes = [_vp, _vp, _vp, _vp, _vp, _i32, _i32, _vp]
_lib.chain_draft_step.restype = C.c_int
_lib.chain_draft_step.argtypes = [_vp, _i32, _i64, _i32, _i32, _f32, _vp, _vp, _vp, _vp, _vp, _i32, _i32, _vp, _vp]
_lib.tree_accept_compact.restype = C.c_int
_lib.tree_accept_compact.argtypes = [_vp, _vp, _vp, _vp, _i32, _i32, _vp, _vp, _kvp, _vp, _vp, _vp, _vp,
                                     _vp, _vp]


def _p(t):
    return None if t is None else t.data_ptr()


def _stream(stream=None):
    return (stream or torch.cuda.current_stream()).cuda_stream


def _check(code: int):
    if code != 0:
        raise TwigError(code)


def lib_path() -> str:
    return _LIB_PATH


def twig_set_launch_overlap(on: int) -> int:
    """Programmatic stream serialization for the attention and accept kernels (default on)."""
    return int(_lib.twig_set_launch_overlap(int(on)))


def twig_workspace_bytes(batch, n_q_heads, head_dim, max_len, max_nodes) -> int:
    return int(_lib.twig_workspace_bytes(batch, n_q_heads, head_dim, max_len, max_nodes))


def tree_attention_workspace_bytes(batch, n_q_heads, max_nodes) -> int:
    """Scratch of the persistent attention kernel: zero-filled at first use, passed to no other call."""
    return int(_lib.tree_attention_workspace_bytes(batch, n_q_heads, max_nodes))


def ttp_score(twig_q, twig_k, prefix_len, vis_start, n_vis, scores, ws, norm_scope=0,
              softmax_scale=0.0, dev_status=None, stream=None):
    """twig_q [B,Hq,d], twig_k [B,Hkv,Lmax,d] bf16; scores [B,m_max] fp32 (out)."""
    B, Hq, d = twig_q.shape
    _check(_lib.ttp_score(_p(twig_q), _p(twig_k), twig_k.stride(0), twig_k.stride(1), twig_k.stride(2),
                          twig_k.shape[2], _p(prefix_len), _p(vis_start), _p(n_vis), B, Hq,
                          twig_k.shape[1], d, norm_scope, softmax_scale, _p(scores), scores.shape[1],
                          _p(dev_status), _p(ws), ws.numel() * ws.element_size(), _stream(stream)))


def ttp_score_gated(twig_q, q_gate, twig_k, k_gate, prefix_len, vis_start, n_vis, scores, ws, norm_scope=1,
                    softmax_scale=0.0, dev_status=None, stream=None):
    """ttp_score of (q_gate * twig_q, k_gate * twig_k), element-wise products formed in the kernel;
    q_gate like twig_q, k_gate with twig_k's shape and strides."""
    B, Hq, d = twig_q.shape
    assert q_gate.shape == twig_q.shape and q_gate.is_contiguous()
    assert k_gate.shape == twig_k.shape and k_gate.stride() == twig_k.stride()
    _check(_lib.ttp_score_gated(_p(twig_q), _p(q_gate), _p(twig_k), _p(k_gate), twig_k.stride(0), twig_k.stride(1),
                                twig_k.stride(2), twig_k.shape[2], _p(prefix_len), _p(vis_start), _p(n_vis), B, Hq,
                                twig_k.shape[1], d, norm_scope, softmax_scale, _p(scores), scores.shape[1],
                                _p(dev_status), _p(ws), ws.numel() * ws.element_size(), _stream(stream)))


def ttp_multiquery_workspace_bytes(batch, n_q_heads, n_text_max, m_max, k_max_len):
    return int(_lib.ttp_multiquery_workspace_bytes(batch, n_q_heads, n_text_max, m_max, k_max_len))


def ttp_score_multiquery(q_text, twig_k, prefix_len, vis_start, n_vis, scores, ws, softmax_scale=0.0,
                         dev_status=None, stream=None):
    """q_text [B,Hq,Nmax,d] (the text tokens after the image, in order), twig_k [B,Hkv,Lmax,d] bf16;
    scores [B,m_max] fp32 (out): attention from those tokens to every visual token, summed over
    tokens, averaged over heads."""
    B, Hq, N, d = q_text.shape
    assert q_text.is_contiguous()
    _check(_lib.ttp_score_multiquery(_p(q_text), N, _p(twig_k), twig_k.stride(0), twig_k.stride(1), twig_k.stride(2),
                                     twig_k.shape[2], _p(prefix_len), _p(vis_start), _p(n_vis), B, Hq, twig_k.shape[1],
                                     d, softmax_scale, _p(scores), scores.shape[1], _p(dev_status), _p(ws),
                                     ws.numel() * ws.element_size(), _stream(stream)))


def ttp_score_noalloc(twig_q, twig_k, prefix_len, vis_start, n_vis, scores, norm_scope=0,
                      softmax_scale=0.0, dev_status=None, stream=None):
    """ttp_score for callers that may not allocate device memory: the logits scratch is a fixed
    NOALLOC_SCRATCH_BYTES array inside the library (shared by all calls on the device, so calls
    that overlap on the GPU race).  Raises TwigError(TWIG_ERR_WORKSPACE) when
    batch * n_q_heads * prompt length does not fit."""
    B, Hq, d = twig_q.shape
    _check(_lib.ttp_score_noalloc(_p(twig_q), _p(twig_k), twig_k.stride(0), twig_k.stride(1),
                                  twig_k.stride(2), twig_k.shape[2], _p(prefix_len), _p(vis_start),
                                  _p(n_vis), B, Hq, twig_k.shape[1], d, norm_scope, softmax_scale,
                                  _p(scores), scores.shape[1], _p(dev_status), _stream(stream)))


def ttp_topk(scores, n_vis, keep, kept_idx, dev_status=None, stream=None):
    """scores [B,m_max] fp32; kept_idx [B,r_max] int32 (out, ascending, -1 padded)."""
    _check(_lib.ttp_topk(_p(scores), _p(n_vis), _p(keep), scores.shape[0], scores.shape[1],
                         kept_idx.shape[1], _p(kept_idx), _p(dev_status), _stream(stream)))


def ttp_compact(src: KV, dst: KV, kept_idx, keep, prefix_len, vis_start, n_vis, pos_in=None,
                pos_out=None, new_len=None, dev_status=None, stream=None):
    pos_stride = pos_in.shape[1] if pos_in is not None else 0
    _check(_lib.ttp_compact(C.byref(src), C.byref(dst), _p(kept_idx), kept_idx.shape[1], _p(keep),
                            _p(prefix_len), _p(vis_start), _p(n_vis), _p(pos_in), _p(pos_out),
                            pos_stride, _p(new_len), _p(dev_status), _stream(stream)))


def ttp_compact_rows(src, dst, kept_idx, keep, prefix_len, vis_start, n_vis, new_len=None, dev_status=None,
                     stream=None):
    """Prune a [B, L, width] token sequence (e.g. layer-K hidden states): dst[b, j] = src[b, idx_b[j]].
    src/dst: CUDA tensors whose last dimension is contiguous and a multiple of 16 bytes."""
    es = src.element_size()
    assert src.dim() == 3 and dst.dim() == 3 and src.stride(2) == 1 and dst.stride(2) == 1
    _check(_lib.ttp_compact_rows(_p(src), _p(dst), src.shape[2] * es, src.stride(1) * es, src.stride(0) * es,
                                 src.shape[1], dst.stride(1) * es, dst.stride(0) * es, dst.shape[1], src.shape[0],
                                 _p(kept_idx), kept_idx.shape[1], _p(keep), _p(prefix_len), _p(vis_start),
                                 _p(n_vis), _p(new_len), _p(dev_status), _stream(stream)))


def ttp_score_topk_compact(twig_q, twig_k, prefix_len, vis_start, n_vis, keep, scores, kept_idx,
                           src: KV, dst: KV, ws, pos_in=None, pos_out=None, new_len=None,
                           norm_scope=0, softmax_scale=0.0, dev_status=None, stream=None):
    pos_stride = pos_in.shape[1] if pos_in is not None else 0
    _check(_lib.ttp_score_topk_compact(
        _p(twig_q), _p(twig_k), twig_k.stride(0), twig_k.stride(1), twig_k.stride(2), twig_k.shape[2],
        _p(prefix_len), _p(vis_start), _p(n_vis), _p(keep), twig_q.shape[1], norm_scope, softmax_scale,
        _p(scores), scores.shape[1], _p(kept_idx), kept_idx.shape[1], C.byref(src), C.byref(dst),
        _p(pos_in), _p(pos_out), pos_stride, _p(new_len), _p(dev_status), _p(ws),
        ws.numel() * ws.element_size(), _stream(stream)))


def tree_verify_attention(q, tree_k, tree_v, cache: KV, layer, kv_len, n_nodes, parent, out, lse=None,
                          softmax_scale=0.0, dev_status=None, ws=None, stream=None, flags=None):
    """q/out [B,T,Hq,d]; tree_k/v [B,Hkv,T,d]; parent [B,T] int32; lse [B,Hq,T] fp32 or None.
    ws: scratch of the persistent kernel (zero-filled at first use, this call's only) or None.
    flags: None calls tree_verify_attention, an int (see attn_flags) tree_verify_attention_ex."""
    B, T, Hq, d = q.shape
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    args = (_p(q), _p(tree_k), _p(tree_v), C.byref(cache), layer, _p(kv_len), _p(n_nodes), _p(parent), T, Hq,
            softmax_scale, _p(out), _p(lse), _p(dev_status), _p(ws), ws_bytes, _stream(stream))
    if flags is None:
        _check(_lib.tree_verify_attention(*args))
    else:
        _check(_lib.tree_verify_attention_ex(*args, int(flags)))


def tree_verify_attention_ex(q, tree_k, tree_v, cache: KV, layer, kv_len, n_nodes, parent, out, flags, lse=None,
                             softmax_scale=0.0, dev_status=None, ws=None, stream=None):
    """tree_verify_attention with the per-call flags word (see attn_flags)."""
    tree_verify_attention(q, tree_k, tree_v, cache, layer, kv_len, n_nodes, parent, out, lse=lse,
                          softmax_scale=softmax_scale, dev_status=dev_status, ws=ws, stream=stream, flags=int(flags))


class TreeState:
    """Device arrays of the token trees under construction: node_tok / node_parent (int32) and
    node_score (fp32), [batch, cap] each."""

    def __init__(self, batch, cap, device):
        self.batch, self.cap = batch, cap
        self.tok = torch.empty((batch, cap), dtype=torch.int32, device=device)
        self.parent = torch.empty((batch, cap), dtype=torch.int32, device=device)
        self.score = torch.empty((batch, cap), dtype=torch.float32, device=device)
        self.ticket = torch.zeros((batch,), dtype=torch.int32, device=device)    # tree_grow_level's counters


def tree_reset(state: TreeState, stream=None):
    _check(_lib.tree_reset(_p(state.tok), _p(state.parent), _p(state.score), state.cap, state.batch, _stream(stream)))


def tree_expand_level(logits, src_node, n_children, level_base, state: TreeState, dev_status=None, stream=None):
    """logits [B, rows, V] bf16 or fp32 (last dim contiguous); src_node [B, rows] int32 (-1: unused row)."""
    B, rows, V = logits.shape
    assert logits.stride(2) == 1 and logits.stride(0) == rows * logits.stride(1)
    _check(_lib.tree_expand_level(_p(logits), 1 if logits.dtype == torch.float32 else 0, logits.stride(1), V, rows,
                                  _p(src_node), n_children, level_base, _p(state.tok), _p(state.parent), _p(state.score),
                                  state.cap, B, _p(dev_status), _stream(stream)))


def tree_select_expansion(state: TreeState, level_lo, level_hi, expand_node, dev_status=None, stream=None):
    """expand_node [B, K] int32 (out): the K best nodes of level_lo..level_hi-1, ascending, -1 padded."""
    _check(_lib.tree_select_expansion(_p(state.score), state.cap, level_lo, level_hi, expand_node.shape[1],
                                      _p(expand_node), state.batch, _p(dev_status), _stream(stream)))


def tree_finalize(state: TreeState, n_built, n_max, parent, draft_tok, n_nodes, kept_node=None, dev_status=None,
                  stream=None):
    """parent, draft_tok [B, t_max], n_nodes [B] int32 (out): the pruned trees in verification layout."""
    _check(_lib.tree_finalize(_p(state.tok), _p(state.parent), _p(state.score), state.cap, n_built, n_max, _p(parent),
                              _p(draft_tok), _p(n_nodes), _p(kept_node), parent.shape[1], state.batch, _p(dev_status),
                              _stream(stream)))


def tree_grow_level(logits, src_node, n_children, level_base, state: TreeState, expand_node=None, n_max=0, parent=None,
                    draft_tok=None, n_nodes=None, kept_node=None, dev_status=None, stream=None):
    """One level in one launch: the expansion, then either the next level's expansion nodes
    (expand_node [B, K] given) or the final pruning to n_max nodes (parent, draft_tok, n_nodes given)."""
    B, rows, V = logits.shape
    assert logits.stride(2) == 1 and logits.stride(0) == rows * logits.stride(1)
    n_select = expand_node.shape[1] if expand_node is not None else 0
    t_max = parent.shape[1] if parent is not None else 0
    _check(_lib.tree_grow_level(_p(logits), 1 if logits.dtype == torch.float32 else 0, logits.stride(1), V, rows,
                                _p(src_node), n_children, level_base, _p(state.tok), _p(state.parent), _p(state.score),
                                state.cap, B, n_select, _p(expand_node), n_max, _p(parent), _p(draft_tok), _p(n_nodes),
                                _p(kept_node), t_max, _p(state.ticket), _p(dev_status), _stream(stream)))


def tree_base_argmax(logits, n_nodes, base_argmax, dev_status=None, stream=None):
    """logits [B, T, V] bf16 or fp32 (last dim contiguous); base_argmax [B, T] int32 (out):
    the target's greedy token after every tree node, lowest index on ties."""
    B, T, V = logits.shape
    assert logits.stride(2) == 1 and logits.stride(0) == T * logits.stride(1)
    _check(_lib.tree_base_argmax(_p(logits), 1 if logits.dtype == torch.float32 else 0, logits.stride(1), V,
                                 _p(n_nodes), B, T, _p(base_argmax), _p(dev_status), _stream(stream)))


def chain_draft_reset(parent, draft_tok, n_nodes, active, tok_prob=None, stream=None):
    """Start a drafting iteration: every request holds its root only and is drafting."""
    _check(_lib.chain_draft_reset(_p(parent), _p(draft_tok), _p(tok_prob), _p(n_nodes), _p(active), parent.shape[1],
                                  parent.shape[0], _stream(stream)))


def chain_draft_step(logits, max_draft, threshold, parent, draft_tok, n_nodes, active, tok_prob=None, dev_status=None,
                     stream=None):
    """logits [B, V] bf16 or fp32 (last dim contiguous): one draft distribution per request.  Appends the
    greedy token to the chains of the requests that are still drafting and applies the early exit."""
    B, V = logits.shape
    assert logits.stride(1) == 1
    _check(_lib.chain_draft_step(_p(logits), 1 if logits.dtype == torch.float32 else 0, logits.stride(0), V, max_draft,
                                 threshold, _p(parent), _p(draft_tok), _p(tok_prob), _p(n_nodes), _p(active),
                                 parent.shape[1], B, _p(dev_status), _stream(stream)))


def tree_accept_compact(parent, draft_tok, base_argmax, n_nodes, tree_k_all, tree_v_all, cache: KV,
                        kv_len, accept_len, path, bonus_tok, dev_status=None, stream=None):
    """tree_k_all/v_all [Nl,B,Hkv,T,d]; path [B,d_max] int32 (out)."""
    _check(_lib.tree_accept_compact(_p(parent), _p(draft_tok), _p(base_argmax), _p(n_nodes),
                                    parent.shape[1], path.shape[1], _p(tree_k_all), _p(tree_v_all),
                                    C.byref(cache), _p(kv_len), _p(accept_len), _p(path), _p(bonus_tok),
                                    _p(dev_status), _stream(stream)))
