"""CPU oracle for one PosS speculative round.  TEST INFRASTRUCTURE ONLY.

A plain, slow numpy restatement of what the path computes, written from the
paper (PosS: position specialists for speculative decoding) and from the
readings listed in the design notes.  It shares no code with the CUDA library
and must never be imported by the product path: only the tests, the smoke
check and the benchmark's CPU-baseline leg may call it.

Numerics.  ``Num(dtype, act)``: all arithmetic runs in ``dtype`` (float64 by
default, float32 for the full-size workloads where memory and time matter).
``act == "bf16"`` reproduces the precision contract of the bf16 path: the
activation operand of every matrix product, and every value stored in a KV
cache, is rounded to bfloat16 first; everything else (residual stream, norms,
softmax, rotary embedding, SiLU, scores) stays in ``dtype``.  ``act == "none"``
is the exact (check-mode) arithmetic.

Parity status: every function here is pinned by tests/test_oracle_pins.py
except the statistics the paper obtains from trained drafters (acceptance
length, speed-up): those need the authors' checkpoints and datasets and are
"parity unpinned".
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np


# --------------------------------------------------------------------------- numerics

def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round to the nearest bfloat16 value (ties to even); result keeps x's dtype."""
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    b = x32.view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(x.dtype if isinstance(x, np.ndarray) else np.float32)


def widen(w: np.ndarray, dtype) -> np.ndarray:
    """Stored parameter -> working precision.  uint16 arrays hold bfloat16 bit patterns."""
    if w.dtype == np.uint16:
        return (w.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(dtype, copy=False)
    return w.astype(dtype, copy=False)


@dataclass
class Num:
    dtype: type = np.float64
    act: str = "none"          # "none" | "bf16"

    def r(self, x: np.ndarray) -> np.ndarray:
        return round_bf16(x) if self.act == "bf16" else x

    def w(self, w: np.ndarray) -> np.ndarray:
        return widen(w, self.dtype)


def linear(x, W, num: Num, b=None):
    """y = x W^T (+ b) with the activation operand rounded per the contract."""
    y = num.r(np.asarray(x, dtype=num.dtype)) @ num.w(W).T
    if b is not None:
        y = y + num.w(b)
    return y


def rmsnorm(x, g, eps, num: Num):
    """RMSNorm: g * x / sqrt(mean(x^2) + eps).  g None = no normalisation at all."""
    if g is None:
        return x
    x = np.asarray(x, dtype=num.dtype)
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps) * num.w(g)


def rope(v, pos, theta, num: Num):
    """Rotary embedding, rotate-half pairing (j, j + d/2), angle pos * theta^(-2j/d).

    v: [rows][heads][d]; pos: [rows] integer positions.
    """
    v = np.asarray(v, dtype=num.dtype)
    d = v.shape[-1]
    half = d // 2
    j = np.arange(half, dtype=np.float64)
    inv = theta ** (-2.0 * j / d)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv[None, :]
    c = np.cos(ang).astype(num.dtype)[:, None, :]
    s = np.sin(ang).astype(num.dtype)[:, None, :]
    a, b = v[..., :half], v[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(x):
    return x / (1.0 + np.exp(-x))


def log_softmax_rows(z):
    m = z.max(axis=-1, keepdims=True)
    return z - (m + np.log(np.exp(z - m).sum(axis=-1, keepdims=True)))


def topk_rows(z, k):
    """Indices of the k largest entries per row, best first; ties -> lowest index."""
    order = np.argsort(-z, axis=-1, kind="stable")
    return order[..., :k]


def topk_by_score(scores, k):
    """Indices of the k best scores, best first; ties -> lower index."""
    order = np.argsort(-np.asarray(scores), kind="stable")
    return order[:k]


# --------------------------------------------------------------------------- specialist schedule

def specialist_for_position(i: int, n: int, S: int) -> int:
    """1-based specialist serving 0-based draft position i: ceil((i+1)/n) (Eq. 7 and its worked
    example: n=2 puts positions 0,1 on specialist 1 and 2,3 on specialist 2), clamped to S when a
    round drafts deeper than S*n positions."""
    return min((i + n) // n, S)


def specialist_param_count(hidden, n_q_heads, n_kv_heads, head_dim, ffn) -> int:
    """Parameters of one specialist = one transformer layer (Section 3.3)."""
    qd, kd = n_q_heads * head_dim, n_kv_heads * head_dim
    return 2 * hidden * qd + 2 * hidden * kd + 3 * hidden * ffn


# --------------------------------------------------------------------------- attention

def masked_attention(q, K, V, visible, scale, num: Num):
    """Definition of the tree attention.

    q [rows][Hq][d]; K, V [Hkv][slots][d]; visible [rows][slots] bool.
    Query head h reads KV head h // (Hq // Hkv).  Returns o [rows][Hq][d].
    """
    rows, Hq, d = q.shape
    Hkv = K.shape[0]
    group = Hq // Hkv
    o = np.zeros((rows, Hq, d), dtype=num.dtype)
    for r in range(rows):
        idx = np.nonzero(visible[r])[0]
        for h in range(Hq):
            kh = h // group
            s = (K[kh, idx, :] @ q[r, h, :]) * scale
            p = np.exp(s - s.max())
            p = p / p.sum()
            o[r, h, :] = p @ V[kh, idx, :]
    return o


def ancestor_matrix(parents) -> np.ndarray:
    """anc[r][j] = True iff j is r or an ancestor of r (parents[root] = -1)."""
    n = len(parents)
    anc = np.zeros((n, n), dtype=bool)
    for r in range(n):
        j = r
        while j >= 0:
            anc[r, j] = True
            j = int(parents[j])
    return anc


def pack_mask(anc: np.ndarray) -> np.ndarray:
    """bool [rows][cols] -> uint64 [rows][ceil(cols/64)], bit j of word j//64."""
    rows, cols = anc.shape
    words = (cols + 63) // 64
    out = np.zeros((rows, words), dtype=np.uint64)
    for r in range(rows):
        for j in np.nonzero(anc[r])[0]:
            out[r, j // 64] |= np.uint64(1) << np.uint64(j % 64)
    return out


def tree_attention(q, kv, prefix_len, parents, scale, num: Num):
    """Standalone tree attention: row r sees cache slots [0, prefix_len) and the tree slots
    prefix_len + j of its ancestors j and of itself.  kv [2][Hkv][cap][d] already holds the
    rows' own keys/values in slots prefix_len .. prefix_len+rows-1."""
    rows = q.shape[0]
    anc = ancestor_matrix(parents)
    vis = np.zeros((rows, prefix_len + rows), dtype=bool)
    vis[:, :prefix_len] = True
    vis[:, prefix_len:] = anc
    K = num.w(kv[0])[:, :prefix_len + rows]
    V = num.w(kv[1])[:, :prefix_len + rows]
    return masked_attention(num.r(np.asarray(num.w(q), dtype=num.dtype)), K, V, vis, scale, num)


# --------------------------------------------------------------------------- decoder layer pieces

def kv_project(h0, lw, pos, cfg, num: Num):
    """Keys/values of rows whose layer input is h0: norm -> Wk/Wv -> rotary on k -> cache precision."""
    xn = rmsnorm(h0, lw["norm_in"], cfg.rms_eps, num)
    rows = h0.shape[0]
    k = linear(xn, lw["wk"], num).reshape(rows, cfg.n_kv_heads, cfg.head_dim)
    v = linear(xn, lw["wv"], num).reshape(rows, cfg.n_kv_heads, cfg.head_dim)
    k = rope(k, pos, cfg.rope_theta, num)
    return num.r(k), num.r(v)


def q_project(h0, lw, pos, cfg, num: Num):
    xn = rmsnorm(h0, lw["norm_in"], cfg.rms_eps, num)
    rows = h0.shape[0]
    q = linear(xn, lw["wq"], num).reshape(rows, cfg.n_q_heads, cfg.head_dim)
    return num.r(rope(q, pos, cfg.rope_theta, num))


def layer_tail(h0, o, lw, cfg, num: Num):
    """Everything after attention: h1 = h0 + Wo o;  y = h1 + Wdown(silu(Wgate u) * (Wup u)), u = norm(h1)."""
    rows = h0.shape[0]
    h1 = h0 + linear(o.reshape(rows, -1), lw["wo"], num)
    u = rmsnorm(h1, lw["norm_post"], cfg.rms_eps, num)
    act = silu(linear(u, lw["w_gate"], num)) * linear(u, lw["w_up"], num)
    return h1 + linear(act, lw["w_down"], num)


def fc_input(tok, feat, w, lw, num: Num):
    """EAGLE-style layer input (Eq. 1): fc([token embedding ; feature]) (+ bias)."""
    emb = num.w(w["embed"][np.asarray(tok, dtype=np.int64)])
    x = np.concatenate([emb, np.asarray(feat, dtype=num.dtype)], axis=-1)
    return linear(x, lw["fc_w"], num, lw.get("fc_b"))


# --------------------------------------------------------------------------- draft round

@dataclass
class Node:
    tok: int
    feat_in: np.ndarray          # feature half of this node's input pair
    level: int                   # 0 = root / verified pair
    slot: int                    # KV slot in every specialist's cache
    pos: int                     # rotary position
    parent: "Node | None" = None
    cand: int = -1               # flat candidate index (-1 for verified pairs)
    score: float = 0.0
    fout: np.ndarray | None = None


@dataclass
class StepTrace:
    specialist: int                      # 0-based
    frontier_cand: list                  # flat candidate index per current row (-1 = root)
    n_rows: int                          # rows in the fc / KV projection batch (pending + current)
    fout: np.ndarray                     # [Mc][H]
    logits: np.ndarray | None            # [Mc][V] (kept only when asked)
    top_ids: np.ndarray                  # [Mc][K]
    top_logp: np.ndarray                 # [Mc][K]
    row_margin: np.ndarray               # [Mc] smallest logit gap that decides this row's top-K list
    own_top_ids: np.ndarray | None = None  # the oracle's own top-K ids (differs from top_ids only when following)
    frontier_margin: float = math.inf    # gap between the last kept and first dropped candidate score
    own_frontier: np.ndarray | None = None  # flat candidate indices the oracle itself would expand next
    next_frontier: np.ndarray | None = None  # flat candidate indices actually expanded next


@dataclass
class DraftResult:
    tokens: np.ndarray           # [n_nodes] node 0 = root
    parents: np.ndarray          # [n_nodes] parents[0] = -1
    scores: np.ndarray           # [n_nodes] cumulative log-prob, root 0
    depth: np.ndarray            # [n_nodes]
    anc_mask: np.ndarray         # [n_nodes][words] uint64
    n_nodes: int
    cand_tok: np.ndarray
    cand_parent: np.ndarray      # flat index of the parent candidate, -1 = root
    cand_score: np.ndarray
    cand_level: np.ndarray
    selected: np.ndarray         # flat candidate indices kept by the rerank, ascending
    rerank_margin: float
    steps: list = field(default_factory=list)


def _decision_margin(sorted_vals, k):
    """Smallest adjacent gap among the first k+1 entries of a descending list (what a
    perturbation must overcome to change the ordered top-k)."""
    v = np.asarray(sorted_vals[: k + 1], dtype=np.float64)
    if len(v) < 2:
        return math.inf
    return float(np.min(v[:-1] - v[1:]))


def draft_round(cfg, w, draft_kv, prefix_len, new_tokens, new_features, depth, topk, total,
                num: Num, linearize=False, keep_logits=False, follow=None):
    """One PosS draft phase (Eq. 9 applied position by position, tree drafting with
    width / depth / total tokens as in Section 4.1).

    draft_kv: array [S][2][Hkv][cap][d] in working precision, slots [0, prefix_len) valid for
    every specialist; slots from prefix_len on are written here.  new_tokens/new_features are the
    verified pairs not yet in any cache; the last one is the root pair [x_t ; f_{t-1}].

    follow: replay of another implementation's decisions, every value still computed here:
    follow["top_ids"][i] the [Mc][K] token ids of step i's candidates, follow["frontier"][i] the flat
    candidate indices expanded at step i+1, follow["selected"] the rerank's choice.  Optional teacher
    forcing of values, so that a comparison is per step and rounding noise does not pile up over
    the depth: follow["features"][i] ([Mc][H]) replaces this step's output features as the input of
    the children, and follow["cand_scores"] (flat) replaces the parents' cumulative scores.
    With follow["force_head_input"] the forced feature of step i is also what this step's LM head reads, so
    the head stage is checked on identical inputs while the feature itself is compared separately (a
    feature of magnitude 16..64 has a bf16 spacing of 2^-4..2^-2: two features that agree to 1e-2
    still round differently in a few percent of their elements, which moves logits of magnitude ~70
    by more than any fixed absolute tolerance).
    """
    S, n, K = cfg.S, cfg.n, topk
    H = cfg.hidden
    n_new = len(new_tokens)
    scale = 1.0 / math.sqrt(cfg.head_dim)
    tree_base = prefix_len + n_new
    root_pos = tree_base - 1

    verified = [Node(int(new_tokens[j]), np.asarray(widen(new_features[j], num.dtype)), 0,
                     prefix_len + j, prefix_len + j) for j in range(n_new)]
    root = verified[-1]
    levels = [[root]]                       # levels[l] = frontier nodes of level l
    cached = [set() for _ in range(S)]      # id(node) whose K/V specialist s already holds

    cand_tok, cand_parent, cand_score, cand_level, cand_node_parent = [], [], [], [], []
    steps = []

    for i in range(depth):
        s = specialist_for_position(i, n, S) - 1
        lw = w["spec"][s]
        current = levels[i]
        earlier = verified + [nd for lv in levels[1:i] for nd in lv]
        pending = [nd for nd in earlier if id(nd) not in cached[s] and all(nd is not c for c in current)]
        batch = pending + current
        toks = [nd.tok for nd in batch]
        feats = np.stack([nd.feat_in for nd in batch])
        pos = np.array([nd.pos for nd in batch])
        h0 = fc_input(toks, feats, w, lw, num)
        k, v = kv_project(h0, lw, pos, cfg, num)
        for r, nd in enumerate(batch):
            draft_kv[s, 0, :, nd.slot, :] = k[r]
            draft_kv[s, 1, :, nd.slot, :] = v[r]
            cached[s].add(id(nd))
        Mc = len(current)
        h0c = h0[-Mc:]
        q = q_project(h0c, lw, pos[-Mc:], cfg, num)

        if not linearize:
            cap = draft_kv.shape[3]
            vis = np.zeros((Mc, cap), dtype=bool)
            vis[:, :tree_base] = True
            for r, nd in enumerate(current):
                a = nd
                while a is not None and a.level >= 1:
                    vis[r, a.slot] = True
                    a = a.parent
            o = masked_attention(q, draft_kv[s, 0], draft_kv[s, 1], vis, scale, num)
        else:
            # definition by Eq. 9: the specialist runs over the node's own linearised history
            o = np.zeros((Mc, cfg.n_q_heads, cfg.head_dim), dtype=num.dtype)
            for r, nd in enumerate(current):
                path = []
                a = nd
                while a is not None and a.level >= 1:
                    path.append(a)
                    a = a.parent
                path = verified + path[::-1]
                ph0 = fc_input([p.tok for p in path], np.stack([p.feat_in for p in path]), w, lw, num)
                pk, pv = kv_project(ph0, lw, np.array([p.pos for p in path]), cfg, num)
                Kseq = np.concatenate([draft_kv[s, 0][:, :prefix_len], pk.transpose(1, 0, 2)], axis=1)
                Vseq = np.concatenate([draft_kv[s, 1][:, :prefix_len], pv.transpose(1, 0, 2)], axis=1)
                vis1 = np.ones((1, Kseq.shape[1]), dtype=bool)
                o[r] = masked_attention(q[r:r + 1], Kseq, Vseq, vis1, scale, num)[0]

        fout = layer_tail(h0c, num.r(o), lw, cfg, num)
        forced_f = None if follow is None or "features" not in follow else np.asarray(follow["features"][i], dtype=num.dtype)
        for r, nd in enumerate(current):
            nd.fout = fout[r] if forced_f is None else forced_f[r]
        head_in = forced_f if forced_f is not None and follow.get("force_head_input") else fout
        logits = linear(head_in, w["lm_head"], num)
        logp = log_softmax_rows(logits)
        own_ids = topk_rows(logits, K)
        srt = -np.sort(-logits, axis=-1)
        row_margin = np.array([_decision_margin(srt[r], K) for r in range(Mc)])
        top_ids = own_ids if follow is None else np.asarray(follow["top_ids"][i])
        top_logp = np.take_along_axis(logp, top_ids, axis=-1)

        base = len(cand_tok)
        for r, nd in enumerate(current):
            for kk in range(K):
                cand_tok.append(int(top_ids[r, kk]))
                cand_parent.append(nd.cand)
                cand_node_parent.append(nd)
                cand_score.append(nd.score + top_logp[r, kk])
                cand_level.append(i + 1)

        st = StepTrace(s, [nd.cand for nd in current], len(batch), fout,
                       logits if keep_logits else None, top_ids, top_logp, row_margin, own_ids)
        if i < depth - 1:
            step_scores = np.array(cand_score[base:])
            own_pick = topk_by_score(step_scores, K)
            pick = own_pick if follow is None else np.asarray(follow["frontier"][i]) - base
            st.own_frontier = own_pick + base
            st.next_frontier = np.asarray(pick) + base
            ss = -np.sort(-step_scores)
            st.frontier_margin = _decision_margin(ss, min(K, len(ss)))
            nxt = []
            for jj, c in enumerate(pick):
                par = cand_node_parent[base + c]
                sc = cand_score[base + c]
                if follow is not None and "cand_scores" in follow:
                    sc = float(follow["cand_scores"][base + int(c)])
                nxt.append(Node(cand_tok[base + c], par.fout, i + 1, tree_base + i * K + jj,
                                root_pos + i + 1, par, base + int(c), sc))
            levels.append(nxt)
        steps.append(st)

    # a round shallower than the specialist schedule still leaves every cache complete
    for s in range(S):
        todo = [nd for nd in verified if id(nd) not in cached[s]]
        if todo:
            lw = w["spec"][s]
            h0 = fc_input([nd.tok for nd in todo], np.stack([nd.feat_in for nd in todo]), w, lw, num)
            k, v = kv_project(h0, lw, np.array([nd.pos for nd in todo]), cfg, num)
            for r, nd in enumerate(todo):
                draft_kv[s, 0, :, nd.slot, :] = k[r]
                draft_kv[s, 1, :, nd.slot, :] = v[r]

    res = rerank(np.array(cand_tok), np.array(cand_parent), np.array(cand_score, dtype=np.float64),
                 np.array(cand_level), int(root.tok), total,
                 selected=None if follow is None else follow.get("selected"))
    res.steps = steps
    return res


def draft_round_batched(cfg, w, draft_kvs, prefix_lens, new_tokens, new_features, depth, topk, total, num: Num):
    """Drafting for several independent sequences in one call: by definition every sequence is drafted on its own
    (its own caches, prefix length and verified pairs); nothing couples them.  Speed is measured as throughput
    against vanilla decoding (Section 4.1), which is what batching the sequences serves."""
    return [draft_round(cfg, w, draft_kvs[b], prefix_lens[b], new_tokens[b], new_features[b], depth, topk, total, num)
            for b in range(len(draft_kvs))]


def rerank(cand_tok, cand_parent, cand_score, cand_level, root_tok, total, selected=None) -> DraftResult:
    """Keep the `total` best candidates by cumulative log-prob (ties -> lower flat index), list them
    in creation order behind the root, remap parents, and build the packed ancestor masks."""
    n_cand = len(cand_tok)
    keep = min(total, n_cand)
    order = topk_by_score(cand_score, n_cand)
    if selected is None:
        sel = np.sort(order[:keep])
    else:
        sel = np.sort(np.asarray(selected))
    srt = cand_score[order]
    margin = float(srt[keep - 1] - srt[keep]) if keep < n_cand else math.inf
    new_index = {-1: 0}
    for j, c in enumerate(sel):
        new_index[int(c)] = j + 1
    n_nodes = len(sel) + 1
    tokens = np.zeros(n_nodes, dtype=np.int32)
    parents = np.full(n_nodes, -1, dtype=np.int32)
    scores = np.zeros(n_nodes, dtype=np.float64)
    depth = np.zeros(n_nodes, dtype=np.int32)
    tokens[0] = root_tok
    for j, c in enumerate(sel):
        tokens[j + 1] = cand_tok[c]
        parents[j + 1] = new_index[int(cand_parent[c])]
        scores[j + 1] = cand_score[c]
        depth[j + 1] = cand_level[c]
    mask = pack_mask(ancestor_matrix(parents))
    return DraftResult(tokens, parents, scores, depth, mask, n_nodes, np.asarray(cand_tok),
                       np.asarray(cand_parent), np.asarray(cand_score), np.asarray(cand_level), sel, margin)


# --------------------------------------------------------------------------- target model

def target_forward(cfg, w, target_kv, prefix_len, tokens, positions, parents, num: Num):
    """Target rows under a tree mask.  Row r is written to cache slot prefix_len + r, sits at rotary
    position positions[r], and sees slots [0, prefix_len) plus its ancestors and itself.
    A chain (parents = -1, 0, 1, ...) is ordinary causal decoding.

    target_kv: [layers][2][Hkv][cap][d] working precision.  Returns (features [rows][H] after the
    final norm, logits [rows][V])."""
    rows = len(tokens)
    scale = 1.0 / math.sqrt(cfg.head_dim)
    anc = ancestor_matrix(parents)
    vis = np.zeros((rows, prefix_len + rows), dtype=bool)
    vis[:, :prefix_len] = True
    vis[:, prefix_len:] = anc
    pos = np.asarray(positions)
    x = num.w(w["embed"][np.asarray(tokens, dtype=np.int64)]).astype(num.dtype)
    for li, lw in enumerate(w["target"]):
        k, v = kv_project(x, lw, pos, cfg, num)
        target_kv[li, 0, :, prefix_len:prefix_len + rows, :] = k.transpose(1, 0, 2)
        target_kv[li, 1, :, prefix_len:prefix_len + rows, :] = v.transpose(1, 0, 2)
        q = q_project(x, lw, pos, cfg, num)
        o = masked_attention(q, target_kv[li, 0][:, :prefix_len + rows], target_kv[li, 1][:, :prefix_len + rows],
                             vis, scale, num)
        x = layer_tail(x, num.r(o), lw, cfg, num)
    feat = rmsnorm(x, w["final_norm"], cfg.rms_eps, num)
    logits = linear(feat, w["lm_head"], num)
    return feat, logits


def chain_parents(rows):
    return np.arange(-1, rows - 1, dtype=np.int32)


def argmax_rows(z):
    """Row argmax, ties -> lowest index."""
    return np.argmax(z, axis=-1).astype(np.int32)


def new_target_kv(cfg, capacity, num: Num):
    return np.zeros((cfg.n_target_layers, 2, cfg.n_kv_heads, capacity, cfg.head_dim), dtype=num.dtype)


def plain_greedy(cfg, w, prompt, n_generate, num: Num):
    """Vanilla autoregressive greedy decoding of the target: the definition of the lossless output."""
    cap = len(prompt) + n_generate + 1
    kv = new_target_kv(cfg, cap, num)
    n = len(prompt)
    feat, logits = target_forward(cfg, w, kv, 0, prompt, np.arange(n), chain_parents(n), num)
    out = [int(argmax_rows(logits[-1:])[0])]
    P = n
    while len(out) < n_generate:
        feat, logits = target_forward(cfg, w, kv, P, [out[-1]], [P], chain_parents(1), num)
        out.append(int(argmax_rows(logits)[0]))
        P += 1
    return np.array(out[:n_generate], dtype=np.int32)


# --------------------------------------------------------------------------- verification

def accept_walk(tokens, parents, g):
    """Greedy acceptance: starting at the root, move to the child whose token equals the target's
    greedy token at the current node; stop when no child matches.  Acceptance of position i implies
    acceptance of every earlier position (A_i subset of A_{i-1}).
    Returns (path node indices incl. root, n_accepted = len(path) - 1, bonus token)."""
    cur = 0
    path = [0]
    while True:
        nxt = -1
        for c in range(len(tokens)):
            if parents[c] == cur and tokens[c] == g[cur]:
                nxt = c
                break
        if nxt < 0:
            break
        cur = nxt
        path.append(cur)
    return path, len(path) - 1, int(g[cur])


def verify_accept(target_logits, target_features, tokens, parents):
    """Row argmax of the target logits, accept walk, and the verified pairs handed to the next draft
    round: [token at path[k+1] ; target feature at path[k]] for k < a, then [bonus ; feature at path[a]]."""
    g = argmax_rows(np.asarray(target_logits))
    path, a, bonus = accept_walk(tokens, parents, g)
    new_tokens = [int(tokens[path[k + 1]]) for k in range(a)] + [bonus]
    new_features = np.stack([target_features[path[k]] for k in range(a + 1)])
    return path, a, bonus, np.array(new_tokens, dtype=np.int32), new_features


def sample_walk(target_logits, tokens, parents, temperature, uniforms, with_residual=False):
    """Verification at a temperature > 0 (the second acceptance setting of Section 5; the rejection-sampling
    phase of Section 2.1): the emitted tokens must be distributed as the target's own sampling.  The draft
    tree proposes its candidates deterministically (top-k, no sampling in the drafter), i.e. each candidate is
    a point mass q(x) = 1, for which rejection sampling reads: at the current node with target distribution
    p = softmax(logits / temperature), test the node's children in node order; child x is accepted with
    probability min(1, p(x) / q(x)) = p(x) (u < p(x) for the next uniform u); on rejection the residual
    distribution norm(max(p - q, 0)) = p with p(x) removed and renormalised replaces p and the next child is
    tested; when no child is left, the bonus token is drawn from the current p by inverse CDF (first index
    whose cumulative probability exceeds u).  One uniform per tested child plus one for the bonus, consumed
    in order.  Returns (path incl. root, n_accepted, bonus token, uniforms used) and, with_residual, the
    distribution the bonus was drawn from."""
    z = np.asarray(target_logits, dtype=np.float64)
    cur, path, k = 0, [0], 0
    while True:
        t = z[cur] / float(temperature)
        p = np.exp(t - t.max())
        p /= p.sum()
        nxt = -1
        for c in range(len(tokens)):
            if parents[c] != cur:
                continue
            x = int(tokens[c])
            u = float(uniforms[k])
            k += 1
            if u < p[x]:
                nxt = c
                break
            p[x] = 0.0
            total = p.sum()
            if total <= 0.0:            # the children carried all of the mass: nothing is left to draw from
                p[x] = 1.0
                total = 1.0
            p /= total
        if nxt >= 0:
            cur = nxt
            path.append(cur)
            continue
        u = float(uniforms[k])
        k += 1
        cdf = np.cumsum(p)
        bonus = int(np.searchsorted(cdf, u * cdf[-1], side="right"))
        last = int(np.nonzero(p > 0)[0][-1])
        out = (path, len(path) - 1, min(bonus, last), k)
        return out + (p,) if with_residual else out


@dataclass
class Counters:
    """Per-position acceptance counters: N_i = rounds in which draft position i was accepted."""
    max_depth: int
    rounds: int = 0
    accepted_at: np.ndarray | None = None

    def __post_init__(self):
        if self.accepted_at is None:
            self.accepted_at = np.zeros(self.max_depth + 1, dtype=np.int64)

    def add(self, a: int):
        self.rounds += 1
        self.accepted_at[1:a + 1] += 1

    def pos_acc(self):
        """pos-acc_i = P(A_i | A_{i-1}) = N_i / N_{i-1} (Eq. 3), with A_0 certain so pos-acc_1 = N_1 / R."""
        out = np.full(self.max_depth + 1, np.nan)
        prev = self.rounds
        for i in range(1, self.max_depth + 1):
            if prev > 0:
                out[i] = self.accepted_at[i] / prev
            prev = self.accepted_at[i]
        return out

    def mean_accepted(self):
        return self.accepted_at[1:].sum() / max(self.rounds, 1)


def drafter_prefill(cfg, w, draft_kv, start, tokens, features, num: Num):
    """Fill every specialist's cache with the K/V of verified pairs at slots start .. start+len-1
    (each specialist keeps its own cache; Section 3.3)."""
    pos = np.arange(start, start + len(tokens))
    for s in range(cfg.S):
        lw = w["spec"][s]
        h0 = fc_input(tokens, np.asarray(widen(features, num.dtype)), w, lw, num)
        k, v = kv_project(h0, lw, pos, cfg, num)
        draft_kv[s, 0, :, start:start + len(tokens), :] = k.transpose(1, 0, 2)
        draft_kv[s, 1, :, start:start + len(tokens), :] = v.transpose(1, 0, 2)


def speculative_greedy(cfg, w, prompt, n_generate, num: Num, depth=None, topk=None, total=None, log=None):
    """Full draft-then-verify loop at temperature 0 (Section 2.1): prefill, then rounds of
    draft tree -> tree-masked target pass -> accept walk -> cache commit.  Returns (tokens, Counters)."""
    depth = cfg.depth if depth is None else depth
    topk = cfg.topk if topk is None else topk
    total = cfg.total if total is None else total
    n = len(prompt)
    cap_t = n + n_generate + total + 2 + depth
    tkv = new_target_kv(cfg, cap_t, num)
    dkv = np.zeros((cfg.S, 2, cfg.n_kv_heads, cap_t + (depth - 1) * topk, cfg.head_dim), dtype=num.dtype)
    feat, logits = target_forward(cfg, w, tkv, 0, prompt, np.arange(n), chain_parents(n), num)
    first = int(argmax_rows(logits[-1:])[0])
    out = [first]
    P = n                                   # tokens in the target cache
    # pair j = [token j+1 ; feature j]; pairs 0..n-2 are filled ahead, pair n-1 is the first root
    if n > 1:
        drafter_prefill(cfg, w, dkv, 0, prompt[1:], feat[:-1], num)
    dP = n - 1                              # pairs in every drafter cache
    new_tok = np.array([first], dtype=np.int32)
    new_feat = feat[-1:]
    ctr = Counters(depth)
    while len(out) < n_generate:
        tree = draft_round(cfg, w, dkv, dP, new_tok, new_feat, depth, topk, total, num)
        pos = P + tree.depth
        tf, tl = target_forward(cfg, w, tkv, P, tree.tokens, pos, tree.parents, num)
        path, a, bonus, new_tok, new_feat = verify_accept(tl, tf, tree.tokens, tree.parents)
        for k in range(1, a + 1):            # compaction: accepted tree slots become contiguous
            tkv[:, :, :, P + k, :] = tkv[:, :, :, P + path[k], :]
        dP = P                               # every pair up to the old root is now cached
        P += a + 1
        out.extend(int(t) for t in new_tok)
        ctr.add(a)
        if log is not None:
            log.append((a, path))
    return np.array(out[:n_generate], dtype=np.int32), ctr
