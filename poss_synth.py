"""Seeded synthetic inputs for the PosS speculative-round path.

This module only draws numbers and lays them out; it contains none of the
method's arithmetic.  Both the CPU oracle's tests and the CUDA path's tests /
benchmark take their inputs from here so that the two sides see identical bits.

Every tensor is drawn from its own counter-based stream (numpy Philox keyed by
(seed, tensor name, chunk index)), so a tensor's bits do not depend on which
other tensors were generated, on thread scheduling or on the platform.

Storage conventions
-------------------
* ``dtype == "fp32"``: float32 arrays.
* ``dtype == "bf16"``: uint16 arrays holding bfloat16 bit patterns (values drawn
  in fp32 and rounded once, round-to-nearest-even).  The consumer widens them.

Workload recipes (shapes follow the paper's experiment setup: Llama-3-8B-Instruct
and Llama-2-13B-chat geometry, tree width 10, total tokens 60/80, depth 6/8;
Section 4.1 "Implementations" and Appendix C of the paper):

* every weight matrix, embedding and LM head ~ N(0, 0.02); RMSNorm gains ~ 1 + N(0, 0.1)
  (non-trivial, so that a dropped, misplaced or shifted gain shows in every comparison);
  fc bias ~ N(0, 0.02);
* prefix KV of every specialist ~ N(0, 1); features ~ N(0, 1); token ids uniform.
"""
from __future__ import annotations

import dataclasses
import hashlib
import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import numpy as np

_CHUNK = 1 << 24


@dataclass(frozen=True)
class PossConfig:
    name: str
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    rope_theta: float
    rms_eps: float
    dtype: str              # "fp32" | "bf16"
    S: int                  # number of position specialists
    n: int                  # draft positions per specialist (PosS-n)
    depth: int              # L: drafter steps per round
    topk: int               # K: tree width
    total: int              # T: draft tokens kept after rerank
    prefix: int             # P: committed prefix length for drafter-only workloads
    n_target_layers: int = 0
    fc_bias: bool = True
    norm_in: bool = True    # False: the draft layers carry no input norm (their "norm_in" is None)

    def replace(self, **kw) -> "PossConfig":
        return dataclasses.replace(self, **kw)

    @property
    def n_candidates(self) -> int:
        return self.topk + (self.depth - 1) * self.topk * self.topk

    @property
    def tree_slots(self) -> int:
        return (self.depth - 1) * self.topk


CONFIGS = {
    # tiny fp32 toy with a 4-layer target: full speculative loop, chain drafting
    "c1": PossConfig("c1", 256, 4, 4, 64, 688, 1024, 1.0e4, 1e-5, "fp32", 3, 2, 6, 1, 6, 64, 4),
    # Llama-3-8B-shaped drafter, 6 specialists (PosS-1)
    "c2": PossConfig("c2", 4096, 32, 8, 128, 14336, 128256, 5.0e5, 1e-5, "bf16", 6, 1, 6, 10, 60, 1024),
    # Llama-2-13B-shaped drafter, 3 specialists x 2 positions (PosS-2)
    "c3": PossConfig("c3", 5120, 40, 40, 128, 13824, 32000, 1.0e4, 1e-5, "bf16", 3, 2, 6, 10, 60, 2048),
    # Llama-3-8B shape, long prefix, depth 8, 80 tokens, 4 specialists x 2
    "c4": PossConfig("c4", 4096, 32, 8, 128, 14336, 128256, 5.0e5, 1e-5, "bf16", 4, 2, 8, 10, 80, 8192),
    # full loop: 32-layer target + the c2 drafter
    "c5": PossConfig("c5", 4096, 32, 8, 128, 14336, 128256, 5.0e5, 1e-5, "bf16", 6, 1, 6, 10, 60, 512, 32),
    # small shapes for tests: several tiles, ragged tails, GQA, tree mode
    "t_fp32": PossConfig("t_fp32", 192, 6, 2, 32, 344, 777, 1.0e4, 1e-5, "fp32", 3, 2, 5, 3, 14, 37, 2),
    "t_bf16": PossConfig("t_bf16", 512, 8, 2, 64, 1408, 5000, 1.0e4, 1e-5, "bf16", 3, 2, 6, 4, 24, 300, 2),
    # mid-size bf16: Llama geometry scaled down 4x, many tiles per GEMM, ragged vocab
    "m_bf16": PossConfig("m_bf16", 1024, 8, 2, 128, 3584, 32003, 5.0e5, 1e-5, "bf16", 6, 1, 6, 10, 60, 700, 2),
}


def _key(seed: int, name: str, chunk: int) -> int:
    h = hashlib.blake2b(f"{seed}/{name}/{chunk}".encode(), digest_size=8).digest()
    return int.from_bytes(h, "little")


def _to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bfloat16 bit pattern, round-to-nearest-even (storage format only)."""
    b = x.view(np.uint32)
    return ((b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


def normal(seed: int, name: str, shape, std: float, dtype: str) -> np.ndarray:
    """N(0, std) tensor; float32 for "fp32", uint16 bf16 bits for "bf16"."""
    shape = tuple(int(s) for s in np.atleast_1d(shape))
    total = int(np.prod(shape)) if shape else 1
    out = np.empty(total, dtype=np.float32 if dtype == "fp32" else np.uint16)
    n_chunks = (total + _CHUNK - 1) // _CHUNK

    def work(c: int) -> None:
        lo = c * _CHUNK
        hi = min(total, lo + _CHUNK)
        g = np.random.Generator(np.random.Philox(key=_key(seed, name, c)))
        x = g.standard_normal(hi - lo, dtype=np.float32)
        x *= np.float32(std)
        out[lo:hi] = x if dtype == "fp32" else _to_bf16_bits(x)

    if n_chunks <= 1:
        for c in range(n_chunks):
            work(c)
    else:
        with ThreadPoolExecutor(max(1, min(n_chunks, os.cpu_count() or 1))) as ex:
            list(ex.map(work, range(n_chunks)))
    return out.reshape(shape)


def ones(shape, dtype: str) -> np.ndarray:
    if dtype == "fp32":
        return np.ones(shape, dtype=np.float32)
    return np.full(shape, 0x3F80, dtype=np.uint16)


def gain(seed: int, name: str, shape, dtype: str, spread: float = 0.1) -> np.ndarray:
    """RMSNorm gain 1 + N(0, spread), same storage conventions as normal()."""
    shape = tuple(int(s) for s in np.atleast_1d(shape))
    g = np.random.Generator(np.random.Philox(key=_key(seed, name, 0)))
    x = np.float32(1.0) + np.float32(spread) * g.standard_normal(shape, dtype=np.float32)
    return x if dtype == "fp32" else _to_bf16_bits(x.ravel()).reshape(shape)


def tokens(seed: int, name: str, count: int, vocab: int) -> np.ndarray:
    g = np.random.Generator(np.random.Philox(key=_key(seed, name, 0)))
    return g.integers(0, vocab, size=count, dtype=np.int64).astype(np.int32)


def layer_weights(cfg: PossConfig, seed: int, tag: str, with_fc: bool) -> dict:
    H, F = cfg.hidden, cfg.ffn
    qd, kd = cfg.n_q_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim
    dt = cfg.dtype
    w = {}
    if with_fc:
        # columns [0,H) multiply the token embedding, [H,2H) the feature
        w["fc_w"] = normal(seed, f"{tag}.fc_w", (H, 2 * H), 0.02, dt)
        w["fc_b"] = normal(seed, f"{tag}.fc_b", (H,), 0.02, dt) if cfg.fc_bias else None
    w["norm_in"] = gain(seed, f"{tag}.norm_in", (H,), dt) if (cfg.norm_in or not with_fc) else None
    w["wq"] = normal(seed, f"{tag}.wq", (qd, H), 0.02, dt)
    w["wk"] = normal(seed, f"{tag}.wk", (kd, H), 0.02, dt)
    w["wv"] = normal(seed, f"{tag}.wv", (kd, H), 0.02, dt)
    w["wo"] = normal(seed, f"{tag}.wo", (H, qd), 0.02, dt)
    w["norm_post"] = gain(seed, f"{tag}.norm_post", (H,), dt)
    w["w_gate"] = normal(seed, f"{tag}.w_gate", (F, H), 0.02, dt)
    w["w_up"] = normal(seed, f"{tag}.w_up", (F, H), 0.02, dt)
    w["w_down"] = normal(seed, f"{tag}.w_down", (H, F), 0.02, dt)
    return w


def make_weights(cfg: PossConfig, seed: int, alias_specialists: bool = False) -> dict:
    """Embedding, LM head, S specialist layers and (if any) the target's layers.

    ``alias_specialists`` makes every specialist the same object (one weight
    set used S times): the single-draft-layer baseline the paper calls PosS-inf.
    """
    w = {
        "embed": normal(seed, "embed", (cfg.vocab, cfg.hidden), 0.02, cfg.dtype),
        "lm_head": normal(seed, "lm_head", (cfg.vocab, cfg.hidden), 0.02, cfg.dtype),
    }
    if alias_specialists:
        one = layer_weights(cfg, seed, "spec0", True)
        w["spec"] = [one for _ in range(cfg.S)]
    else:
        w["spec"] = [layer_weights(cfg, seed, f"spec{j}", True) for j in range(cfg.S)]
    w["target"] = [layer_weights(cfg, seed, f"tgt{j}", False) for j in range(cfg.n_target_layers)]
    w["final_norm"] = gain(seed, "final_norm", (cfg.hidden,), cfg.dtype)
    return w


def draft_kv_capacity(cfg: PossConfig, max_new: int) -> int:
    return cfg.prefix + max_new + cfg.tree_slots


def make_draft_kv(cfg: PossConfig, seed: int, capacity: int, prefix_len: int | None = None) -> np.ndarray:
    """Per-specialist KV caches [S][2][Hkv][capacity][d]; first prefix_len slots ~ N(0,1), rest 0."""
    P = cfg.prefix if prefix_len is None else prefix_len
    dt = cfg.dtype
    kv = np.zeros((cfg.S, 2, cfg.n_kv_heads, capacity, cfg.head_dim),
                  dtype=np.float32 if dt == "fp32" else np.uint16)
    if P > 0:
        kv[:, :, :, :P, :] = normal(seed, "draft_kv", (cfg.S, 2, cfg.n_kv_heads, P, cfg.head_dim), 1.0, dt)
    return kv


def make_round_inputs(cfg: PossConfig, seed: int, n_new: int = 1):
    """Verified (token, feature) pairs handed to a draft round; the last one is the root."""
    toks = tokens(seed, "new_tokens", n_new, cfg.vocab)
    feats = normal(seed, "new_features", (n_new, cfg.hidden), 1.0, cfg.dtype)
    return toks, feats


def make_prompt(cfg: PossConfig, seed: int, count: int) -> np.ndarray:
    return tokens(seed, "prompt", count, cfg.vocab)


def make_attention_case(seed: int, rows: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                        prefix_len: int, capacity: int, dtype: str):
    """Standalone tree-attention inputs: q [rows][Hq][d], kv [2][Hkv][capacity][d] ~ N(0,1)."""
    q = normal(seed, "attn_q", (rows, n_q_heads, head_dim), 1.0, dtype)
    kv = np.zeros((2, n_kv_heads, capacity, head_dim), dtype=np.float32 if dtype == "fp32" else np.uint16)
    kv[:, :, :prefix_len + rows, :] = normal(seed, "attn_kv", (2, n_kv_heads, prefix_len + rows, head_dim), 1.0, dtype)
    return q, kv


def random_tree_parents(seed: int, rows: int, max_children: int = 3) -> np.ndarray:
    """parents[r] < r for r >= 1, parents[0] = -1: a random tree in parent-before-child order."""
    g = np.random.Generator(np.random.Philox(key=_key(seed, "tree", 0)))
    parents = np.full(rows, -1, dtype=np.int32)
    n_children = np.zeros(rows, dtype=np.int64)
    for r in range(1, rows):
        while True:
            p = int(g.integers(0, r))
            if n_children[p] < max_children:
                break
        parents[r] = p
        n_children[p] += 1
    return parents


def make_mimic_weights(cfg: PossConfig, seed: int) -> dict:
    """A drafter that imitates a ONE-layer target, so that speculative rounds accept several tokens.

    Every specialist aliases the target's single layer and its fc keeps only the token-embedding
    half of the input pair (fc_w = [I | 0], no bias).  The drafter then sees the same token stream
    as the target, shifted by one position and without the very first token, and mostly predicts the
    target's own greedy token.  Pure input construction: no arithmetic of the method happens here.
    """
    assert cfg.n_target_layers == 1
    w = make_weights(cfg, seed)
    H = cfg.hidden
    if cfg.dtype == "fp32":
        fc = np.zeros((H, 2 * H), dtype=np.float32)
        fc[np.arange(H), np.arange(H)] = 1.0
        fb = np.zeros((H,), dtype=np.float32)
    else:
        fc = np.zeros((H, 2 * H), dtype=np.uint16)
        fc[np.arange(H), np.arange(H)] = 0x3F80
        fb = np.zeros((H,), dtype=np.uint16)
    one = dict(w["target"][0])
    one["fc_w"] = fc
    one["fc_b"] = fb
    w["spec"] = [one for _ in range(cfg.S)]
    return w
