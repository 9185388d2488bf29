"""Thin ctypes binding of libposs.so: argument marshalling only.

PyTorch provides device memory and streams; every step of the path runs in the library's kernels.
There is no fallback: if the library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libposs.so")

POSS_FP32, POSS_BF16 = 0, 1
POSS_MAX_ROWS, POSS_MAX_TOPK, POSS_MAX_DEPTH = 128, 16, 16
PROF_KINDS = ("fc", "qkv", "attention", "o", "gate_up", "down", "lm_head")
POSS_OPT_ATTENTION_TCGEN05, POSS_OPT_SWIGLU_IN_KERNEL = 0, 1
KERNEL_NAMES = {0: "other", 1: "gather_x", 2: "embed_rows", 3: "rmsnorm", 4: "reduce_norm", 5: "rope_append",
                6: "attn_tc", 7: "attn_mma", 8: "attn_combine_bf16", 9: "attn_partial", 10: "attn_combine",
                11: "splitk_reduce", 12: "splitk_swiglu", 13: "silu_mul", 14: "cast", 15: "gemm_simt",
                16: "topk_partial", 17: "topk_merge", 18: "topk_merge_expand", 19: "argmax_partial", 20: "rerank",
                21: "accept_walk", 22: "sample_walk", 23: "kv_compact", 24: "chain_mask", 25: "tile_contrib",
                32: "gemm_fc", 33: "gemm_qkv", 34: "gemm_o", 35: "gemm_gate_up", 36: "gemm_down", 37: "gemm_lm_head",
                38: "gemm_other"}
STATUS = {0: "POSS_OK", 1: "POSS_E_INVALID", 2: "POSS_E_SHAPE", 3: "POSS_E_CAPACITY", 4: "POSS_E_WORKSPACE",
          5: "POSS_E_CUDA", 6: "POSS_E_TIMEOUT"}


class PossError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: {STATUS.get(code, code)}")
        self.code = code


class poss_config(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("hidden", "n_q_heads", "n_kv_heads", "head_dim", "ffn", "vocab")] + \
               [("rope_theta", C.c_float), ("rms_eps", C.c_float)] + \
               [(n, C.c_int) for n in ("dtype", "n_specialists", "positions_per_specialist", "max_depth", "max_topk",
                                       "max_total", "draft_kv_slots", "n_target_layers", "target_kv_slots", "max_batch")]


LAYER_FIELDS = ("fc_w", "fc_b", "norm_in", "wq", "wk", "wv", "wo", "norm_post", "w_gate", "w_up", "w_down")


class poss_layer_w(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in LAYER_FIELDS]


class poss_weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("target_final_norm", C.c_void_p),
                ("h_specialist", C.POINTER(poss_layer_w)), ("h_target", C.POINTER(poss_layer_w))]


EXPORTS = {
    "poss_workspace_bytes": (C.c_size_t, [C.POINTER(poss_config)]),
    "poss_init": (C.c_int, [C.POINTER(C.c_void_p), C.POINTER(poss_config), C.POINTER(poss_weights), C.c_void_p,
                            C.c_size_t, C.c_void_p]),
    "poss_destroy": (C.c_int, [C.c_void_p]),
    "poss_reset": (C.c_int, [C.c_void_p, C.c_void_p]),
    "poss_draft_prefill": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]),
    "poss_draft_round": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                   C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                   C.c_void_p]),
    "poss_draft_round_batched": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_void_p), C.POINTER(C.c_int), C.c_void_p,
                                           C.c_void_p, C.POINTER(C.c_int), C.c_int, C.c_int, C.c_int, C.c_void_p,
                                           C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "poss_draft_trace": (C.c_int, [C.c_void_p] * 8),
    "poss_draft_trace_seq": (C.c_int, [C.c_void_p, C.c_int] + [C.c_void_p] * 7),
    "poss_tree_attention": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                      C.c_float, C.c_void_p, C.c_void_p]),
    "poss_verify_accept": (C.c_int, [C.c_void_p] * 6 + [C.c_int] + [C.c_void_p] * 6),
    "poss_verify_sample": (C.c_int, [C.c_void_p] * 5 + [C.c_int, C.c_float, C.c_void_p, C.c_int] + [C.c_void_p] * 7),
    "poss_target_forward": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "poss_target_verify": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                     C.c_void_p, C.c_void_p, C.c_void_p]),
    "poss_target_prefill": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p,
                                      C.c_void_p]),
    "poss_kv_compact": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]),
    "poss_get_counters": (C.c_int, [C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.c_void_p]),
    "poss_last_status": (C.c_int, [C.c_void_p, C.c_void_p]),
    "poss_linear": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                              C.c_void_p, C.c_int, C.c_void_p]),
    "poss_lm_head_topk": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                    C.c_void_p]),
    "poss_profile": (C.c_int, [C.c_void_p, C.c_int]),
    "poss_profile_read": (C.c_int, [C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_float)]),
    "poss_timeline_read": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_int32), C.POINTER(C.c_int64),
                                     C.POINTER(C.c_int), C.c_void_p]),
    "poss_attention_plan": (C.c_int, [C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]),
    "poss_launch_count": (C.c_int64, [C.c_void_p]),
    "poss_debug_lose_load": (C.c_int, [C.c_void_p, C.c_int]),
    "poss_debug_option": (C.c_int, [C.c_void_p, C.c_int, C.c_int]),
    "poss_tree_attention_noalloc": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                              C.c_int, C.c_int, C.c_void_p, C.c_float, C.c_void_p, C.c_void_p]),
}

_lib = None


def load_library() -> C.CDLL:
    """Loads libposs.so and declares every exported prototype.  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} not built; run python -m paper_2506_03566_b200.build")
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def _ptr(t) -> int | None:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device pointers must come from contiguous CUDA tensors"
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(code: int, where: str) -> None:
    if code != 0:
        raise PossError(code, where)


def to_device(a: np.ndarray | None, device="cuda"):
    """numpy array from the input generator -> CUDA tensor (uint16 arrays are bfloat16 bit patterns)."""
    if a is None:
        return None
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def make_config(cfg, draft_kv_slots: int, target_kv_slots: int = 0, max_depth=None, max_topk=None,
                max_total=None, max_batch: int = 1) -> poss_config:
    """cfg: any object with the model fields of the synthetic PossConfig."""
    return poss_config(cfg.hidden, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.ffn, cfg.vocab,
                       float(cfg.rope_theta), float(cfg.rms_eps), POSS_BF16 if cfg.dtype == "bf16" else POSS_FP32,
                       cfg.S, cfg.n, max_depth or cfg.depth, max_topk or cfg.topk, max_total or cfg.total,
                       int(draft_kv_slots), cfg.n_target_layers, int(max(target_kv_slots, 1)), int(max_batch))


class Poss:
    """A library context plus the device tensors it borrows (weights, workspace)."""

    def __init__(self, config: poss_config, weights: dict):
        """weights: {"embed", "lm_head", "final_norm", "spec": [layer dict]*S, "target": [layer dict]*n}
        of CUDA tensors (or numpy arrays, which are uploaded)."""
        self.lib = load_library()
        self.config = config
        self.dtype = torch.bfloat16 if config.dtype == POSS_BF16 else torch.float32
        up = lambda v: to_device(v) if isinstance(v, np.ndarray) else v
        cache = {}

        def up_layer(l):
            if id(l) not in cache:          # aliased specialists share one upload
                cache[id(l)] = {k: up(v) for k, v in l.items()}
            return cache[id(l)]

        self.w = {"embed": up(weights["embed"]), "lm_head": up(weights["lm_head"]),
                  "final_norm": up(weights.get("final_norm")),
                  "spec": [up_layer(l) for l in weights["spec"]],
                  "target": [up_layer(l) for l in weights.get("target", [])]}

        def pack(layers):
            arr = (poss_layer_w * max(len(layers), 1))()
            for i, l in enumerate(layers):
                for f in LAYER_FIELDS:
                    setattr(arr[i], f, _ptr(l.get(f)))
            return arr

        self._spec = pack(self.w["spec"])
        self._tgt = pack(self.w["target"])
        pw = poss_weights(_ptr(self.w["embed"]), _ptr(self.w["lm_head"]), _ptr(self.w["final_norm"]),
                          self._spec, self._tgt)
        nbytes = self.lib.poss_workspace_bytes(C.byref(config))
        if nbytes == 0:
            raise PossError(1, "poss_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        ctx = C.c_void_p()
        _check(self.lib.poss_init(C.byref(ctx), C.byref(config), C.byref(pw), _ptr(self.workspace), nbytes, _stream()),
               "poss_init")
        self.ctx = ctx

    def close(self):
        if getattr(self, "ctx", None):
            self.lib.poss_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- allocation helpers (torch owns the memory)
    def new_draft_kv(self):
        c = self.config
        return torch.zeros(c.n_specialists, 2, c.n_kv_heads, c.draft_kv_slots, c.head_dim, dtype=self.dtype,
                           device="cuda")

    def new_target_kv(self):
        c = self.config
        return torch.zeros(c.n_target_layers, 2, c.n_kv_heads, c.target_kv_slots, c.head_dim, dtype=self.dtype,
                           device="cuda")

    # ---- the C calls, same names
    def poss_reset(self):
        _check(self.lib.poss_reset(self.ctx, _stream()), "poss_reset")

    def poss_draft_prefill(self, draft_kv, start, tokens, features):
        n = int(tokens.numel())
        _check(self.lib.poss_draft_prefill(self.ctx, _ptr(draft_kv), start, _ptr(tokens), _ptr(features), n, _stream()),
               "poss_draft_prefill")

    def poss_draft_round(self, draft_kv, prefix_len, new_tokens, new_features, depth, topk, total, out=None):
        """Returns dict of device tensors: tokens, parents, scores, depth, anc_mask, n_nodes."""
        n_new = int(new_tokens.numel())
        if out is None:
            words = (total + 1 + 63) // 64
            dev = "cuda"
            out = {"tokens": torch.empty(total + 1, dtype=torch.int32, device=dev),
                   "parents": torch.empty(total + 1, dtype=torch.int32, device=dev),
                   "scores": torch.empty(total + 1, dtype=torch.float32, device=dev),
                   "depth": torch.empty(total + 1, dtype=torch.int32, device=dev),
                   "anc_mask": torch.empty((total + 1, words), dtype=torch.int64, device=dev),
                   "n_nodes": torch.empty(1, dtype=torch.int32, device=dev)}
        _check(self.lib.poss_draft_round(self.ctx, _ptr(draft_kv), prefix_len, _ptr(new_tokens), _ptr(new_features),
                                         n_new, depth, topk, total, _ptr(out["tokens"]), _ptr(out["parents"]),
                                         _ptr(out["scores"]), _ptr(out["depth"]), _ptr(out["anc_mask"]),
                                         _ptr(out["n_nodes"]), _stream()), "poss_draft_round")
        return out

    def poss_draft_round_batched(self, draft_kvs, prefix_lens, new_tokens, new_features, n_news, depth, topk, total,
                                 out=None):
        """draft_kvs: list of per-sequence cache tensors; prefix_lens, n_news: lists of ints; new_tokens /
        new_features: the sequences' verified pairs one after the other.  Returns dict of device tensors with a
        leading batch dimension."""
        B = len(draft_kvs)
        if out is None:
            words = (total + 1 + 63) // 64
            dev = "cuda"
            out = {"tokens": torch.empty((B, total + 1), dtype=torch.int32, device=dev),
                   "parents": torch.empty((B, total + 1), dtype=torch.int32, device=dev),
                   "scores": torch.empty((B, total + 1), dtype=torch.float32, device=dev),
                   "depth": torch.empty((B, total + 1), dtype=torch.int32, device=dev),
                   "anc_mask": torch.empty((B, total + 1, words), dtype=torch.int64, device=dev),
                   "n_nodes": torch.empty(B, dtype=torch.int32, device=dev)}
        kvp = (C.c_void_p * B)(*[_ptr(k) for k in draft_kvs])
        pl = (C.c_int * B)(*[int(p) for p in prefix_lens])
        nn = (C.c_int * B)(*[int(n) for n in n_news])
        _check(self.lib.poss_draft_round_batched(self.ctx, B, kvp, pl, _ptr(new_tokens), _ptr(new_features), nn, depth,
                                                 topk, total, _ptr(out["tokens"]), _ptr(out["parents"]),
                                                 _ptr(out["scores"]), _ptr(out["depth"]), _ptr(out["anc_mask"]),
                                                 _ptr(out["n_nodes"]), _stream()), "poss_draft_round_batched")
        return out

    def poss_draft_trace(self, depth, topk, n_nodes, seq=None):
        H = self.config.hidden
        nc = topk + (depth - 1) * topk * topk
        dev = "cuda"
        t = {"cand_tokens": torch.empty(nc, dtype=torch.int32, device=dev),
             "cand_parents": torch.empty(nc, dtype=torch.int32, device=dev),
             "cand_scores": torch.empty(nc, dtype=torch.float32, device=dev),
             "frontier": torch.empty((max(depth - 1, 1), topk), dtype=torch.int32, device=dev),
             "step_features": torch.zeros((depth, topk, H), dtype=torch.float32, device=dev),
             "selected": torch.empty(max(n_nodes - 1, 1), dtype=torch.int32, device=dev)}
        if seq is None:
            _check(self.lib.poss_draft_trace(self.ctx, _ptr(t["cand_tokens"]), _ptr(t["cand_parents"]),
                                             _ptr(t["cand_scores"]), _ptr(t["frontier"]), _ptr(t["step_features"]),
                                             _ptr(t["selected"]), _stream()), "poss_draft_trace")
        else:
            _check(self.lib.poss_draft_trace_seq(self.ctx, int(seq), _ptr(t["cand_tokens"]), _ptr(t["cand_parents"]),
                                                 _ptr(t["cand_scores"]), _ptr(t["frontier"]), _ptr(t["step_features"]),
                                                 _ptr(t["selected"]), _stream()), "poss_draft_trace_seq")
        return t

    def poss_tree_attention(self, q, kv, prefix_len, anc_mask, scale, out=None):
        rows = q.shape[0]
        if out is None:
            out = torch.empty_like(q)
        _check(self.lib.poss_tree_attention(self.ctx, _ptr(q), _ptr(kv), kv.shape[2], prefix_len, rows,
                                            _ptr(anc_mask), float(scale), _ptr(out), _stream()), "poss_tree_attention")
        return out

    def poss_verify_accept(self, target_logits, target_argmax, target_features, tokens, parents, rows):
        dev = "cuda"
        H = self.config.hidden
        out = {"path": torch.empty(POSS_MAX_DEPTH + 1, dtype=torch.int32, device=dev),
               "n_accepted": torch.empty(1, dtype=torch.int32, device=dev),
               "bonus": torch.empty(1, dtype=torch.int32, device=dev),
               "new_tokens": torch.zeros(POSS_MAX_DEPTH + 1, dtype=torch.int32, device=dev),
               "new_features": torch.zeros((POSS_MAX_DEPTH + 1, H), dtype=self.dtype, device=dev)}
        _check(self.lib.poss_verify_accept(self.ctx, _ptr(target_logits), _ptr(target_argmax), _ptr(target_features),
                                           _ptr(tokens), _ptr(parents), rows, _ptr(out["path"]),
                                           _ptr(out["n_accepted"]), _ptr(out["bonus"]), _ptr(out["new_tokens"]),
                                           _ptr(out["new_features"]), _stream()), "poss_verify_accept")
        return out

    def poss_verify_sample(self, target_logits, target_features, tokens, parents, rows, temperature, uniforms):
        dev = "cuda"
        H = self.config.hidden
        out = {"path": torch.empty(POSS_MAX_DEPTH + 1, dtype=torch.int32, device=dev),
               "n_accepted": torch.empty(1, dtype=torch.int32, device=dev),
               "bonus": torch.empty(1, dtype=torch.int32, device=dev),
               "new_tokens": torch.zeros(POSS_MAX_DEPTH + 1, dtype=torch.int32, device=dev),
               "new_features": torch.zeros((POSS_MAX_DEPTH + 1, H), dtype=self.dtype, device=dev),
               "uniforms_used": torch.empty(1, dtype=torch.int32, device=dev)}
        _check(self.lib.poss_verify_sample(self.ctx, _ptr(target_logits), _ptr(target_features), _ptr(tokens),
                                           _ptr(parents), rows, float(temperature), _ptr(uniforms),
                                           int(uniforms.numel()), _ptr(out["path"]), _ptr(out["n_accepted"]),
                                           _ptr(out["bonus"]), _ptr(out["new_tokens"]), _ptr(out["new_features"]),
                                           _ptr(out["uniforms_used"]), _stream()), "poss_verify_sample")
        return out

    def poss_target_forward(self, target_kv, prefix_len, tokens, depth, anc_mask, rows, want_logits=False):
        dev = "cuda"
        c = self.config
        feats = torch.empty((rows, c.hidden), dtype=self.dtype, device=dev)
        arg = torch.empty(rows, dtype=torch.int32, device=dev)
        logits = torch.empty((rows, c.vocab), dtype=torch.float32, device=dev) if want_logits else None
        _check(self.lib.poss_target_forward(self.ctx, _ptr(target_kv), prefix_len, _ptr(tokens), _ptr(depth),
                                            _ptr(anc_mask), rows, _ptr(feats), _ptr(arg), _ptr(logits), _stream()),
               "poss_target_forward")
        return feats, arg, logits

    def poss_target_verify(self, target_kv, prefix_len, tokens, depth, anc_mask, rows):
        c = self.config
        feats = torch.empty((rows, c.hidden), dtype=self.dtype, device="cuda")
        arg = torch.empty(rows, dtype=torch.int32, device="cuda")
        _check(self.lib.poss_target_verify(self.ctx, _ptr(target_kv), prefix_len, _ptr(tokens), _ptr(depth),
                                           _ptr(anc_mask), rows, _ptr(feats), _ptr(arg), _stream()),
               "poss_target_verify")
        return feats, arg

    def poss_target_prefill(self, target_kv, start, tokens):
        n = int(tokens.numel())
        feats = torch.empty((n, self.config.hidden), dtype=self.dtype, device="cuda")
        arg = torch.empty(n, dtype=torch.int32, device="cuda")
        _check(self.lib.poss_target_prefill(self.ctx, _ptr(target_kv), start, _ptr(tokens), n, _ptr(feats), _ptr(arg),
                                            _stream()), "poss_target_prefill")
        return feats, arg

    def poss_kv_compact(self, target_kv, prefix_len, path, n_accepted):
        _check(self.lib.poss_kv_compact(self.ctx, _ptr(target_kv), prefix_len, _ptr(path), _ptr(n_accepted), _stream()),
               "poss_kv_compact")

    def poss_get_counters(self):
        r = C.c_int64()
        acc = (C.c_int64 * (POSS_MAX_DEPTH + 2))()
        _check(self.lib.poss_get_counters(self.ctx, C.byref(r), acc, _stream()), "poss_get_counters")
        return r.value, list(acc)[: self.config.max_depth + 1]

    def poss_last_status(self) -> int:
        return self.lib.poss_last_status(self.ctx, _stream())

    def poss_linear(self, x, w, bias=None, residual=None, impl=0):
        M, K = x.shape
        N = w.shape[0]
        out = torch.empty((M, N), dtype=torch.float32, device="cuda")
        _check(self.lib.poss_linear(self.ctx, _ptr(x), M, _ptr(w), N, K, _ptr(bias), _ptr(residual), _ptr(out), impl,
                                    _stream()), "poss_linear")
        return out

    def poss_lm_head_topk(self, features, topk, want_logits=False):
        rows = features.shape[0]
        ids = torch.empty((rows, topk), dtype=torch.int32, device="cuda")
        logp = torch.empty((rows, topk), dtype=torch.float32, device="cuda")
        logits = torch.empty((rows, self.config.vocab), dtype=torch.float32, device="cuda") if want_logits else None
        _check(self.lib.poss_lm_head_topk(self.ctx, _ptr(features), rows, topk, _ptr(ids), _ptr(logp), _ptr(logits),
                                          _stream()), "poss_lm_head_topk")
        return ids, logp, logits

    def poss_profile(self, mode):
        _check(self.lib.poss_profile(self.ctx, int(mode)), "poss_profile")

    def poss_profile_read(self):
        """-> {kind name: (launches, total ms)}"""
        n = (C.c_int * len(PROF_KINDS))()
        ms = (C.c_float * len(PROF_KINDS))()
        _check(self.lib.poss_profile_read(self.ctx, n, ms), "poss_profile_read")
        return {k: (int(n[i]), float(ms[i])) for i, k in enumerate(PROF_KINDS)}

    def poss_timeline_read(self, capacity: int = 8192):
        """-> list of (kernel name, device time in ns) in time order (poss_profile mode 3)."""
        k = (C.c_int32 * capacity)()
        t = (C.c_int64 * capacity)()
        n = C.c_int()
        _check(self.lib.poss_timeline_read(self.ctx, capacity, k, t, C.byref(n), _stream()), "poss_timeline_read")
        rec = sorted(((int(t[i]), int(k[i])) for i in range(n.value)))
        return [(KERNEL_NAMES.get(kk, str(kk)), tt) for tt, kk in rec]

    def poss_debug_lose_load(self, launches: int):
        _check(self.lib.poss_debug_lose_load(self.ctx, int(launches)), "poss_debug_lose_load")

    def poss_debug_option(self, option: int, value: int):
        _check(self.lib.poss_debug_option(self.ctx, int(option), int(value)), "poss_debug_option")

    def poss_launch_count(self) -> int:
        return int(self.lib.poss_launch_count(self.ctx))


def poss_tree_attention_noalloc(q, kv, prefix_len, anc_mask, scale, out):
    """Context-free tree attention for callers that may not allocate device memory: the caller passes
    every buffer, `out` included, and the library keeps its partial results in a fixed internal array.
    q, out [rows][Hq][d]; kv [2][Hkv][slots][d]; anc_mask int64/uint64 [rows][ceil(rows/64)]."""
    lib = load_library()
    rows, hq, d = q.shape
    dtype = POSS_BF16 if q.dtype == torch.bfloat16 else POSS_FP32
    _check(lib.poss_tree_attention_noalloc(_ptr(q), _ptr(kv), kv.shape[2], prefix_len, rows, hq, kv.shape[1], d,
                                           dtype, _ptr(anc_mask), float(scale), _ptr(out), _stream()),
           "poss_tree_attention_noalloc")
    return out
