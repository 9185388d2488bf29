"""Pins for the CPU oracle: each test ties a part of oracle/poss_oracle.py to something other
than itself -- a library implementation of the Llama layer (HF transformers, torch SDPA), facts the
paper states, brute force on tiny inputs, or an invariant the method guarantees."""
import json
import math
import os

import numpy as np
import pytest
import torch

import poss_synth as ps
from oracle import poss_oracle as po

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_facts.json")
NUM = po.Num()          # float64, exact arithmetic


# ----------------------------------------------------------------------------- helpers (library side)

def _t(a):
    return torch.from_numpy(np.asarray(po.widen(a, np.float64), dtype=np.float64))


def hf_model(cfg, w, layers):
    """HF Llama (float64) whose decoder layers carry the given weight dicts."""
    from transformers import LlamaConfig, LlamaForCausalLM
    hc = LlamaConfig(hidden_size=cfg.hidden, intermediate_size=cfg.ffn, num_hidden_layers=len(layers),
                     num_attention_heads=cfg.n_q_heads, num_key_value_heads=cfg.n_kv_heads,
                     head_dim=cfg.head_dim, vocab_size=cfg.vocab, rms_norm_eps=cfg.rms_eps,
                     rope_theta=cfg.rope_theta, attention_bias=False, mlp_bias=False,
                     tie_word_embeddings=False, max_position_embeddings=8192)
    m = LlamaForCausalLM(hc).double().eval()
    sd = {"model.embed_tokens.weight": _t(w["embed"]), "lm_head.weight": _t(w["lm_head"]),
          "model.norm.weight": _t(w["final_norm"])}
    for i, l in enumerate(layers):
        p = f"model.layers.{i}."
        sd[p + "self_attn.q_proj.weight"] = _t(l["wq"])
        sd[p + "self_attn.k_proj.weight"] = _t(l["wk"])
        sd[p + "self_attn.v_proj.weight"] = _t(l["wv"])
        sd[p + "self_attn.o_proj.weight"] = _t(l["wo"])
        sd[p + "mlp.gate_proj.weight"] = _t(l["w_gate"])
        sd[p + "mlp.up_proj.weight"] = _t(l["w_up"])
        sd[p + "mlp.down_proj.weight"] = _t(l["w_down"])
        if l["norm_in"] is None:
            # a layer without an input norm: the library layer with that module taken out
            m.model.layers[i].input_layernorm = torch.nn.Identity()
        else:
            sd[p + "input_layernorm.weight"] = _t(l["norm_in"])
        sd[p + "post_attention_layernorm.weight"] = _t(l["norm_post"])
    missing = m.load_state_dict(sd, strict=False)
    assert not missing.missing_keys and not missing.unexpected_keys
    return m


def hf_layer_out(model, h0):
    """Output of decoder layer 0 (before the model's final norm) for inputs_embeds h0 [rows][H]."""
    grabbed = {}

    def hook(mod, args, out):
        grabbed["y"] = out[0] if isinstance(out, tuple) else out

    h = model.model.layers[0].register_forward_hook(hook)
    with torch.no_grad():
        model(inputs_embeds=torch.from_numpy(h0)[None])
    h.remove()
    return grabbed["y"][0].numpy()


def drafter_chain_by_library(cfg, w, pairs_tok, pairs_feat, depth):
    """Eq. 9 spelled out with library modules: at position i the specialist ceil((i+1)/n) runs as a
    causal one-layer transformer over ALL pairs so far; its last output is the new feature, the LM
    head gives the next token, and [token ; feature] is appended."""
    toks = list(int(t) for t in pairs_tok)
    feats = [np.asarray(f, dtype=np.float64) for f in pairs_feat]
    models = {}
    out_tok, out_logp = [], []
    E = po.widen(w["embed"], np.float64)
    for i in range(depth):
        s = min(math.ceil((i + 1) / cfg.n), cfg.S) - 1
        lw = w["spec"][s]
        if id(lw) not in models:
            models[id(lw)] = hf_model(cfg, w, [lw])
        x = np.concatenate([E[toks], np.stack(feats)], axis=1)
        h0 = torch.nn.functional.linear(torch.from_numpy(x), _t(lw["fc_w"]),
                                        None if lw.get("fc_b") is None else _t(lw["fc_b"])).numpy()
        f = hf_layer_out(models[id(lw)], h0)[-1]
        logp = torch.log_softmax(torch.from_numpy(f) @ _t(w["lm_head"]).T, dim=-1).numpy()
        t = int(np.argmax(logp))
        out_tok.append(t)
        out_logp.append(float(logp[t]))
        toks.append(t)
        feats.append(f)
    return out_tok, out_logp


def fresh_draft_kv(cfg, seed, n_new, num=NUM, prefix=None):
    cap = (cfg.prefix if prefix is None else prefix) + n_new + cfg.tree_slots
    kv = ps.make_draft_kv(cfg, seed, cap, prefix)
    return po.widen(kv, num.dtype).copy()


# ----------------------------------------------------------------------------- facts the paper states

def test_paper_specialist_assignment_example():
    facts = json.load(open(GOLDEN))
    ex = facts["specialist_example_n2"]
    for pos, spec in ex["position_to_specialist"].items():
        assert po.specialist_for_position(int(pos), ex["n"], 99) == spec
    lc = facts["draft_layer_counts_depth6"]
    for n, layers in lc["n_to_layers"].items():
        used = {po.specialist_for_position(i, int(n), 99) for i in range(lc["positions"])}
        assert used == set(range(1, layers + 1))
    # one specialist for all positions = the single-draft-layer baseline
    assert {po.specialist_for_position(i, 6, 1) for i in range(6)} == {1}
    # rounds deeper than S*n stay on the last specialist
    assert po.specialist_for_position(7, 2, 3) == 3


def test_paper_parameter_count():
    facts = json.load(open(GOLDEN))["params_per_specialist_8b"]
    n = po.specialist_param_count(**facts["shape"])
    assert round(n / 1e6) == facts["millions"]
    c2 = ps.CONFIGS["c2"]
    lw = ps.layer_weights(c2.replace(hidden=64, ffn=96, n_q_heads=4, n_kv_heads=2, head_dim=16), 0, "x", False)
    got = sum(v.size for k, v in lw.items() if k.startswith("w"))
    assert got == po.specialist_param_count(64, 4, 2, 16, 96)


def test_synth_configs_follow_paper_knobs():
    facts = json.load(open(GOLDEN))["tree_knobs"]
    for name in ("c2", "c3"):
        c = ps.CONFIGS[name]
        assert (c.topk, c.total, c.depth) == (facts["width"], facts["total"], facts["depth_8b"])
        assert c.S * c.n == c.depth


# ----------------------------------------------------------------------------- primitives vs libraries

def test_bf16_rounding_matches_torch():
    g = np.random.default_rng(0)
    x = np.concatenate([g.standard_normal(5000) * 3, [0.0, 1.0, 1.00390625, 1.01171875, -2.5e-40, 65504.0]])
    want = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(po.round_bf16(x), want)
    bits = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(po.widen(bits, np.float64), want)
    assert np.array_equal(ps._to_bf16_bits(x.astype(np.float32)), bits)


def test_target_forward_matches_hf_llama():
    cfg = ps.CONFIGS["t_fp32"]
    w = ps.make_weights(cfg, 2)
    m = hf_model(cfg, w, w["target"])
    prompt = ps.make_prompt(cfg, 2, 23)
    with torch.no_grad():
        out = m(torch.from_numpy(prompt.astype(np.int64))[None], output_hidden_states=True)
    kv = po.new_target_kv(cfg, 64, NUM)
    feat, logits = po.target_forward(cfg, w, kv, 0, prompt, np.arange(23), po.chain_parents(23), NUM)
    assert np.abs(out.logits[0].numpy() - logits).max() < 1e-6
    assert np.abs(out.hidden_states[-1][0].numpy() - feat).max() < 1e-6
    # incremental decoding through the cache equals the one-shot pass
    kv2 = po.new_target_kv(cfg, 64, NUM)
    po.target_forward(cfg, w, kv2, 0, prompt[:17], np.arange(17), po.chain_parents(17), NUM)
    f2, l2 = po.target_forward(cfg, w, kv2, 17, prompt[17:], np.arange(17, 23), po.chain_parents(6), NUM)
    assert np.abs(l2 - logits[17:]).max() < 1e-9


def test_plain_greedy_matches_hf_generate():
    cfg = ps.CONFIGS["t_fp32"]
    w = ps.make_weights(cfg, 3)
    m = hf_model(cfg, w, w["target"])
    prompt = ps.make_prompt(cfg, 3, 12)
    ids = torch.from_numpy(prompt.astype(np.int64))[None]
    with torch.no_grad():
        g = m.generate(ids, attention_mask=torch.ones_like(ids), max_new_tokens=16, do_sample=False,
                       pad_token_id=0, eos_token_id=None)
    assert np.array_equal(g[0, 12:].numpy(), po.plain_greedy(cfg, w, prompt, 16, NUM))


def test_masked_attention_chain_is_sdpa_causal_with_gqa():
    g = np.random.default_rng(1)
    rows, Hq, Hkv, d, P = 9, 6, 2, 16, 5
    q = g.standard_normal((rows, Hq, d))
    kv = g.standard_normal((2, Hkv, P + rows, d))
    o = po.tree_attention(q, kv, P, po.chain_parents(rows), 1 / math.sqrt(d), NUM)
    # library: SDPA with an explicit mask, KV heads repeated (GQA == MHA with repeated heads)
    K = torch.from_numpy(kv[0]).repeat_interleave(Hq // Hkv, dim=0)
    V = torch.from_numpy(kv[1]).repeat_interleave(Hq // Hkv, dim=0)
    mask = torch.ones(rows, P + rows, dtype=torch.bool)
    mask[:, P:] = torch.tril(torch.ones(rows, rows, dtype=torch.bool))
    want = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q).transpose(0, 1), K, V, attn_mask=mask).transpose(0, 1).numpy()
    assert np.abs(o - want).max() < 1e-12


def test_tree_attention_node_equals_causal_over_its_path_and_ignores_non_ancestors():
    g = np.random.default_rng(2)
    rows, Hq, Hkv, d, P = 14, 4, 2, 8, 6
    parents = ps.random_tree_parents(5, rows)
    q = g.standard_normal((rows, Hq, d))
    kv = g.standard_normal((2, Hkv, P + rows, d))
    scale = 0.37
    o = po.tree_attention(q, kv, P, parents, scale, NUM)
    anc = po.ancestor_matrix(parents)
    for r in range(rows):
        path = [j for j in range(rows) if anc[r, j]]
        assert path[-1] == r
        idx = list(range(P)) + [P + j for j in path]
        K = torch.from_numpy(kv[0][:, idx]).repeat_interleave(Hq // Hkv, dim=0)
        V = torch.from_numpy(kv[1][:, idx]).repeat_interleave(Hq // Hkv, dim=0)
        want = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q[r])[:, None, :], K, V, scale=scale)[:, 0].numpy()
        assert np.abs(o[r] - want).max() < 1e-12
        # perturbing every non-ancestor leaves the row bit-unchanged
        kv2 = kv.copy()
        for j in range(rows):
            if not anc[r, j]:
                kv2[:, :, P + j] += 100.0
        o2 = po.tree_attention(q, kv2, P, parents, scale, NUM)
        assert np.array_equal(o2[r], o[r])


def test_mask_packing():
    parents = np.array([-1, 0, 0, 1, 3, 2] + [5] * 70, dtype=np.int32)
    anc = po.ancestor_matrix(parents)
    m = po.pack_mask(anc)
    assert m.shape == (76, 2)
    for r in range(76):
        for j in range(76):
            assert bool((int(m[r, j // 64]) >> (j % 64)) & 1) == bool(anc[r, j])
    assert int(m[4, 0]) == 0b11011


def test_log_softmax_and_topk():
    g = np.random.default_rng(3)
    z = g.standard_normal((4, 50))
    z[1, 7] = z[1, 30] = z[1].max() + 1.0          # an exact tie: lower index first
    lp = po.log_softmax_rows(z)
    assert np.allclose(np.exp(lp).sum(-1), 1.0, atol=1e-12)
    assert np.allclose(lp, torch.log_softmax(torch.from_numpy(z), -1).numpy(), atol=1e-12)
    ids = po.topk_rows(z, 5)
    for r in range(4):
        full = sorted(range(50), key=lambda j: (-z[r, j], j))
        assert list(ids[r]) == full[:5]
    assert list(ids[1][:2]) == [7, 30]
    assert sorted(po.topk_rows(z, 50)[0]) == list(range(50))
    assert list(po.topk_by_score([1.0, 3.0, 3.0, 2.0], 3)) == [1, 2, 3]


# ----------------------------------------------------------------------------- the draft phase

def test_depth1_is_next_token_prediction_by_a_library_layer():
    """Eq. 2 at k=1 is Eq. 1: one specialist step = a causal one-layer transformer over the pairs."""
    cfg = ps.CONFIGS["t_fp32"].replace(S=1, n=1)
    w = ps.make_weights(cfg, 4)
    toks, feats = ps.make_round_inputs(cfg, 4, n_new=9)
    kv = fresh_draft_kv(cfg, 4, 9, prefix=0)
    res = po.draft_round(cfg, w, kv, 0, toks, feats, 1, 1, 1, NUM)
    want_tok, want_logp = drafter_chain_by_library(cfg, w, toks, feats, 1)
    assert res.n_nodes == 2 and res.tokens[0] == toks[-1]
    assert res.tokens[1] == want_tok[0]
    assert abs(res.scores[1] - want_logp[0]) < 1e-6


@pytest.mark.parametrize("S,n", [(3, 2), (5, 1), (1, 5), (2, 2)])
def test_chain_draft_equals_eq9_with_library_layers(S, n):
    """K=1 chain of depth 5 with DISTINCT specialists: specialist ceil((i+1)/n) (clamped to S)
    re-reads the whole pair history, including features made by earlier specialists."""
    cfg = ps.CONFIGS["t_fp32"].replace(S=S, n=n, depth=5, topk=1, total=5)
    w = ps.make_weights(cfg, 5)
    toks, feats = ps.make_round_inputs(cfg, 5, n_new=4)
    kv = fresh_draft_kv(cfg, 5, 4, prefix=0)
    res = po.draft_round(cfg, w, kv, 0, toks, feats, 5, 1, 5, NUM)
    want_tok, want_logp = drafter_chain_by_library(cfg, w, toks, feats, 5)
    assert list(res.tokens[1:]) == want_tok
    assert list(res.parents) == [-1, 0, 1, 2, 3, 4]
    assert np.abs(res.scores[1:] - np.cumsum(want_logp)).max() < 1e-6
    assert list(res.depth) == [0, 1, 2, 3, 4, 5]


def test_synthetic_gains_are_not_trivial():
    """Every RMSNorm gain of the synthetic recipe differs from 1 (fp32 and bf16 storage alike), element by
    element differently, so that the pins below and every GPU comparison see the gain path."""
    for name in ("t_fp32", "t_bf16"):
        cfg = ps.CONFIGS[name]
        w = ps.make_weights(cfg, 2)
        gains = [w["final_norm"]] + [l[k] for l in w["spec"] + w["target"] for k in ("norm_in", "norm_post")]
        for g in gains:
            g = po.widen(g, np.float64)
            assert g.shape == (cfg.hidden,)
            assert 0.05 < g.std() < 0.2 and abs(g.mean() - 1.0) < 0.05
            assert np.abs(g - np.roll(g, 1)).mean() > 0.05        # a gain read one column off is a different gain
    assert not np.array_equal(w["spec"][0]["norm_in"], w["spec"][1]["norm_in"])
    assert not np.array_equal(w["spec"][0]["norm_in"], w["spec"][0]["norm_post"])


def test_rmsnorm_matches_torch_rms_norm_with_a_gain():
    g = np.random.default_rng(7)
    x = g.standard_normal((5, 48)) * 3.0
    gn = 1.0 + 0.3 * g.standard_normal(48)
    want = torch.nn.functional.rms_norm(torch.from_numpy(x), (48,), torch.from_numpy(gn), 1e-5).numpy()
    assert np.abs(po.rmsnorm(x, gn, 1e-5, NUM) - want).max() < 1e-12
    assert po.rmsnorm(x, None, 1e-5, NUM) is x                    # no norm at all, not a norm with gain 1


@pytest.mark.parametrize("S,n", [(3, 2), (1, 5)])
def test_chain_draft_without_input_norm_equals_the_library_layer_without_it(S, n):
    """Draft layers with norm_in absent: the attention reads fc's output as it is (no normalisation, no gain);
    the library layer with its input_layernorm module removed is the definition."""
    cfg = ps.CONFIGS["t_fp32"].replace(S=S, n=n, depth=5, topk=1, total=5, norm_in=False)
    w = ps.make_weights(cfg, 5)
    assert all(l["norm_in"] is None for l in w["spec"]) and all(l["norm_in"] is not None for l in w["target"])
    toks, feats = ps.make_round_inputs(cfg, 5, n_new=4)
    res = po.draft_round(cfg, w, fresh_draft_kv(cfg, 5, 4, prefix=0), 0, toks, feats, 5, 1, 5, NUM)
    want_tok, want_logp = drafter_chain_by_library(cfg, w, toks, feats, 5)
    assert list(res.tokens[1:]) == want_tok
    assert np.abs(res.scores[1:] - np.cumsum(want_logp)).max() < 1e-6
    # and it is a different function from the normed layer
    w2 = ps.make_weights(cfg.replace(norm_in=True), 5)
    res2 = po.draft_round(cfg, w2, fresh_draft_kv(cfg, 5, 4, prefix=0), 0, toks, feats, 5, 1, 5, NUM)
    assert np.abs(res2.scores[1:] - res.scores[1:]).max() > 1e-4


def test_prefix_cache_equals_recomputing_the_prefix():
    """Slots [0, prefix_len) filled by drafter_prefill behave like pairs processed in the round."""
    cfg = ps.CONFIGS["t_fp32"].replace(topk=2, total=7, depth=4)
    w = ps.make_weights(cfg, 6)
    toks, feats = ps.make_round_inputs(cfg, 6, n_new=8)
    kv_a = fresh_draft_kv(cfg, 6, 8, prefix=0)
    a = po.draft_round(cfg, w, kv_a, 0, toks, feats, 4, 2, 7, NUM)
    kv_b = fresh_draft_kv(cfg, 6, 8, prefix=0)
    po.drafter_prefill(cfg, w, kv_b, 0, toks[:5], feats[:5], NUM)
    b = po.draft_round(cfg, w, kv_b, 5, toks[5:], feats[5:], 4, 2, 7, NUM)
    assert np.array_equal(a.tokens, b.tokens) and np.array_equal(a.parents, b.parents)
    assert np.abs(a.scores - b.scores).max() < 1e-9
    used = 8 + cfg.replace(depth=4, topk=2).tree_slots
    assert np.abs(kv_a[..., :used, :] - kv_b[..., :used, :]).max() < 1e-9


@pytest.mark.parametrize("seed", [7, 8])
def test_batched_pending_rows_equal_linearised_definition(seed):
    """The batched round (pending rows share one projection batch, tree mask) equals running each
    node's specialist over that node's own linearised history."""
    cfg = ps.CONFIGS["t_fp32"]
    w = ps.make_weights(cfg, seed)
    toks, feats = ps.make_round_inputs(cfg, seed, n_new=3)
    ra = po.draft_round(cfg, w, fresh_draft_kv(cfg, seed, 3), cfg.prefix, toks, feats, cfg.depth, cfg.topk, cfg.total, NUM)
    rb = po.draft_round(cfg, w, fresh_draft_kv(cfg, seed, 3), cfg.prefix, toks, feats, cfg.depth, cfg.topk, cfg.total,
                        NUM, linearize=True)
    assert np.array_equal(ra.tokens, rb.tokens) and np.array_equal(ra.parents, rb.parents)
    assert np.abs(ra.scores - rb.scores).max() < 1e-9
    for sa, sb in zip(ra.steps, rb.steps):
        assert np.abs(sa.fout - sb.fout).max() < 1e-9


def test_aliased_specialists_equal_single_draft_layer():
    """S copies of one weight set, any n, reproduce the one-specialist (single draft layer) run."""
    base = ps.CONFIGS["t_fp32"]
    toks, feats = ps.make_round_inputs(base, 9, n_new=2)
    ref = None
    for S, n in [(1, 5), (3, 2), (5, 1)]:
        cfg = base.replace(S=S, n=n)
        w = ps.make_weights(cfg, 9, alias_specialists=True)
        kv = fresh_draft_kv(cfg, 9, 2)
        kv[:] = kv[0:1]                       # identical prefix caches
        r = po.draft_round(cfg, w, kv, cfg.prefix, toks, feats, cfg.depth, cfg.topk, cfg.total, NUM)
        if ref is None:
            ref = r
        else:
            assert np.array_equal(r.tokens, ref.tokens) and np.array_equal(r.parents, ref.parents)
            assert np.abs(r.scores - ref.scores).max() < 1e-9


def _paths(res):
    out = {}
    for r in range(res.n_nodes):
        p, j = [], r
        while j > 0:
            p.append(int(res.tokens[j]))
            j = int(res.parents[j])
        out[tuple(p[::-1])] = r
    return out


@pytest.mark.parametrize("seed", [11, 12])
def test_tree_scores_equal_independent_chain_runs_and_selection_is_valid(seed):
    """Every kept node's score is the sum of log-probs along its token path, each obtained from an
    independent K=1 chain forced along that path; and the tree obeys the selection invariants."""
    cfg = ps.CONFIGS["t_fp32"].replace(vocab=40, depth=4, topk=3, total=12)
    w = ps.make_weights(cfg, seed)
    toks, feats = ps.make_round_inputs(cfg, seed, n_new=2)
    res = po.draft_round(cfg, w, fresh_draft_kv(cfg, seed, 2), cfg.prefix, toks, feats, 4, 3, 12, NUM, keep_logits=True)
    K, L = 3, 4
    assert len(res.cand_tok) == K + (L - 1) * K * K
    assert res.n_nodes == 13
    # structure invariants
    for r in range(1, res.n_nodes):
        p = res.parents[r]
        assert 0 <= p < r                                   # parent listed before child
        assert res.depth[r] == res.depth[p] + 1
        assert res.scores[r] <= res.scores[p] + 1e-15      # log-probs are <= 0
    kept = set(int(c) for c in res.selected)
    for c in kept:                                          # ancestor-closed
        assert res.cand_parent[c] == -1 or int(res.cand_parent[c]) in kept
    worst_kept = min(res.cand_score[c] for c in kept)
    best_dropped = max(res.cand_score[c] for c in range(len(res.cand_tok)) if c not in kept)
    assert worst_kept >= best_dropped
    assert np.array_equal(res.anc_mask, po.pack_mask(po.ancestor_matrix(res.parents)))
    # siblings carry distinct tokens; each step's candidate list per row is the true top-K
    for st in res.steps:
        for r in range(st.top_ids.shape[0]):
            full = sorted(range(cfg.vocab), key=lambda j: (-st.logits[r, j], j))
            assert list(st.top_ids[r]) == full[:K]
    # frontier = K best candidates of the level
    for i, st in enumerate(res.steps[:-1]):
        lvl = [c for c in range(len(res.cand_tok)) if res.cand_level[c] == i + 1]
        best = sorted(lvl, key=lambda c: (-res.cand_score[c], c))[:K]
        assert list(st.next_frontier) == best
    # independent evaluation of every kept path
    for path, r in _paths(res).items():
        if not path:
            continue
        d = len(path)
        forced = {"top_ids": [np.array([[t]]) for t in path], "frontier": [np.array([i]) for i in range(d - 1)]}
        c1 = cfg.replace(topk=1, depth=d, total=d)
        kv = fresh_draft_kv(cfg, seed, 2)       # same prefix bits, capacity for the wider tree
        chain = po.draft_round(c1, w, kv, cfg.prefix, toks, feats, d, 1, d, NUM, follow=forced)
        assert list(chain.tokens[1:]) == list(path)
        assert abs(chain.scores[-1] - res.scores[r]) < 1e-9


def test_round_shallower_than_schedule_still_fills_every_cache():
    cfg = ps.CONFIGS["t_fp32"]
    w = ps.make_weights(cfg, 13)
    toks, feats = ps.make_round_inputs(cfg, 13, n_new=3)
    kv1 = fresh_draft_kv(cfg, 13, 3)
    po.draft_round(cfg, w, kv1, cfg.prefix, toks, feats, 1, 2, 2, NUM)
    kv2 = fresh_draft_kv(cfg, 13, 3)
    po.drafter_prefill(cfg, w, kv2, cfg.prefix, toks, feats, NUM)
    sl = slice(cfg.prefix, cfg.prefix + 3)
    assert np.abs(kv1[:, :, :, sl] - kv2[:, :, :, sl]).max() < 1e-9


# ----------------------------------------------------------------------------- verification

def test_accept_walk_planted_paths():
    parents = ps.random_tree_parents(21, 30)
    g = np.random.default_rng(4)
    tokens = np.zeros(30, dtype=np.int32)
    for p in range(30):                                  # siblings get distinct tokens
        kids = [c for c in range(30) if parents[c] == p]
        tokens[kids] = g.permutation(50)[: len(kids)] + 100
    anc = po.ancestor_matrix(parents)
    for target_node in [0, 7, 29, int(np.argmax(anc.sum(1)))]:
        path = [j for j in range(30) if anc[target_node, j]]
        greedy = np.full(30, 7, dtype=np.int32)          # token 7 is nobody's child token
        for a, b in zip(path[:-1], path[1:]):
            greedy[a] = tokens[b]
        greedy[target_node] = 42
        got_path, a, bonus = po.accept_walk(tokens, parents, greedy)
        assert got_path == path and a == len(path) - 1 and bonus == 42
    feats = g.standard_normal((30, 5))
    logits = g.standard_normal((30, 200))
    path = [j for j in range(30) if anc[29, j]]
    for a_, b_ in zip(path[:-1], path[1:]):
        logits[a_, tokens[b_]] += 12.0
    p2, a2, bonus2, nt, nf = po.verify_accept(logits, feats, tokens, parents)
    assert p2 == path and a2 == len(path) - 1
    assert list(nt[:-1]) == [tokens[j] for j in path[1:]] and nt[-1] == bonus2 == np.argmax(logits[29])
    assert np.array_equal(nf, feats[path])


def test_accept_walk_is_longest_path_matching_teacher_forced_greedy():
    """The accepted path is the longest root path whose tokens equal the target's own greedy
    continuation, computed here by plain step-by-step decoding."""
    cfg = ps.CONFIGS["t_fp32"].replace(n_target_layers=1)
    w = ps.make_mimic_weights(cfg, 15)
    prompt = ps.make_prompt(cfg, 15, 10)
    n = len(prompt)
    kv = po.new_target_kv(cfg, 64, NUM)
    feat, logits = po.target_forward(cfg, w, kv, 0, prompt, np.arange(n), po.chain_parents(n), NUM)
    first = int(np.argmax(logits[-1]))
    dkv = np.zeros((cfg.S, 2, cfg.n_kv_heads, 64, cfg.head_dim))
    po.drafter_prefill(cfg, w, dkv, 0, prompt[1:], feat[:-1], NUM)
    tree = po.draft_round(cfg, w, dkv, n - 1, [first], feat[-1:], cfg.depth, cfg.topk, cfg.total, NUM)
    tf, tl = po.target_forward(cfg, w, kv, n, tree.tokens, n + tree.depth, tree.parents, NUM)
    path, a, bonus = po.accept_walk(tree.tokens, tree.parents, po.argmax_rows(tl))
    cont = po.plain_greedy(cfg, w, np.concatenate([prompt, [first]]), cfg.depth + 1, NUM)
    # brute force: longest tree path matching cont
    best = 0
    for toks_path in _paths(tree):
        d = len(toks_path)
        if list(toks_path) == list(cont[:d]):
            best = max(best, d)
    assert a == best and a >= 1                     # the mimic drafter gets at least one token right
    assert [int(tree.tokens[j]) for j in path[1:]] == list(cont[:a]) and bonus == cont[a]


# ----------------------------------------------------------------------------- verification at temperature > 0

_SW_TOKENS = np.array([9, 2, 5, 0, 3, 1, 4], dtype=np.int32)       # node 0 is the root; siblings differ
_SW_PARENTS = np.array([-1, 0, 0, 0, 1, 1, 2], dtype=np.int32)


def _softmax(z, t):
    e = np.exp(z / t - np.max(z / t))
    return e / e.sum()


def _sample_walk_statistics(walk, n_draws, temperature, seed):
    """Empirical distribution of the first emitted token, and of the second one given the accepted child."""
    g = np.random.default_rng(seed)
    V = 7
    logits = np.random.default_rng(3).standard_normal((7, V)) * 1.5
    first = np.zeros(V)
    second = {c: np.zeros(V) for c in (1, 2, 3)}
    for _ in range(n_draws):
        u = g.random(8)
        path, a, bonus, used = walk(logits, _SW_TOKENS, _SW_PARENTS, temperature, u)
        emitted = [int(_SW_TOKENS[j]) for j in path[1:]] + [bonus]
        assert len(emitted) == a + 1 and 1 <= used <= 8
        first[emitted[0]] += 1
        if a >= 1:
            second[path[1]][emitted[1]] += 1
    return logits, first, second


def _worst_sigma(counts, p):
    """Largest deviation of a frequency from its probability in standard deviations (categories with an expected
    count below 20 are left out: the normal approximation does not hold there)."""
    n = counts.sum()
    keep = n * p >= 20
    return np.max(np.abs(counts[keep] / n - p[keep]) / np.sqrt(p[keep] * (1 - p[keep]) / n))


def test_sample_walk_emits_the_target_distribution():
    """Rejection sampling is lossless: the first emitted token is distributed as softmax(logits[root] / T) whether it
    is an accepted draft token or the bonus, and after an accepted child c the next emitted token is distributed as
    softmax(logits[c] / T).  60,000 draws; every frequency within 4.5 standard deviations."""
    for temperature in (1.0, 0.7):
        logits, first, second = _sample_walk_statistics(po.sample_walk, 60000, temperature, 11)
        assert _worst_sigma(first, _softmax(logits[0], temperature)) < 4.5
        for c, counts in second.items():
            assert counts.sum() > 300
            assert _worst_sigma(counts, _softmax(logits[c], temperature)) < 4.5


def test_the_distribution_pin_catches_a_walk_without_renormalisation():
    """The same statistic must reject a plausible mistake: testing the later siblings against the original
    probabilities instead of the residual distribution."""
    def wrong(target_logits, tokens, parents, temperature, uniforms):
        z = np.asarray(target_logits, dtype=np.float64)
        cur, path, k = 0, [0], 0
        while True:
            p = _softmax(z[cur], temperature)
            nxt = -1
            for c in range(len(tokens)):
                if parents[c] != cur:
                    continue
                u = uniforms[k]; k += 1
                if u < p[int(tokens[c])]:
                    nxt = c
                    break
                p[int(tokens[c])] = 0.0                      # removed, but the rest is not rescaled
            if nxt >= 0:
                cur = nxt; path.append(cur)
                continue
            u = uniforms[k]; k += 1
            cdf = np.cumsum(p)
            return path, len(path) - 1, int(min(np.searchsorted(cdf, u * cdf[-1], side="right"), len(p) - 1)), k
    logits, first, _ = _sample_walk_statistics(wrong, 60000, 1.0, 11)
    assert _worst_sigma(first, _softmax(logits[0], 1.0)) > 8.0


def test_sample_walk_extreme_uniforms_and_uniform_count():
    logits = np.random.default_rng(5).standard_normal((7, 7))
    # u = 0: every tested child is accepted (its probability is positive), the bonus is the first token with mass
    path, a, bonus, used = po.sample_walk(logits, _SW_TOKENS, _SW_PARENTS, 1.0, np.zeros(8))
    assert path == [0, 1, 4] and a == 2 and bonus == 0 and used == 3
    # u just below 1: every child is rejected, the bonus is the last token that still has mass (6; 2, 5, 0 were removed)
    path, a, bonus, used = po.sample_walk(logits, _SW_TOKENS, _SW_PARENTS, 1.0, np.full(8, 1.0 - 1e-12))
    assert path == [0] and a == 0 and bonus == 6 and used == 4
    # first child rejected, second accepted, its only child rejected: 2 + 1 + 1 uniforms
    p0 = _softmax(logits[0], 1.0)
    u = np.array([p0[2] + 1e-9, 0.0, 1.0 - 1e-12, 0.5, 0, 0, 0, 0])
    path, a, bonus, used = po.sample_walk(logits, _SW_TOKENS, _SW_PARENTS, 1.0, u)
    assert path == [0, 2] and a == 1 and used == 4
    p2 = _softmax(logits[2], 1.0)
    p2[4] = 0.0
    assert bonus == int(np.searchsorted(np.cumsum(p2 / p2.sum()), 0.5, side="right"))


def test_sample_walk_at_low_temperature_is_the_greedy_walk():
    """As T -> 0 the target distribution is a point mass on its argmax: a child is accepted iff its token is the
    greedy token, the bonus is the greedy token."""
    parents = ps.random_tree_parents(31, 30)
    g = np.random.default_rng(6)
    tokens = np.zeros(30, dtype=np.int32)
    for p in range(30):
        kids = [c for c in range(30) if parents[c] == p]
        tokens[kids] = g.permutation(50)[: len(kids)] + 100
    anc = po.ancestor_matrix(parents)
    for target_node in (0, 9, 29):
        logits = g.standard_normal((30, 200))
        path = [j for j in range(30) if anc[target_node, j]]
        for a_, b_ in zip(path[:-1], path[1:]):
            logits[a_, tokens[b_]] += 12.0
        logits[target_node, 42] += 12.0
        want = po.accept_walk(tokens, parents, po.argmax_rows(logits))
        got = po.sample_walk(logits, tokens, parents, 0.02, g.uniform(0.001, 0.999, 31))
        assert (got[0], got[1], got[2]) == want


def test_pos_acc_identities():
    c = po.Counters(6)
    g = np.random.default_rng(5)
    accepted = g.integers(0, 7, size=200)
    for a in accepted:
        c.add(int(a))
    N = c.accepted_at
    assert all(N[i] >= N[i + 1] for i in range(1, 6))                 # A_i subset of A_{i-1}
    pa = c.pos_acc()
    assert pa[1] == N[1] / 200
    for k in range(1, 7):                                             # Eq. 4 chain rule
        assert abs(np.prod(pa[1:k + 1]) - N[k] / 200) < 1e-12
        assert N[k] == int((accepted >= k).sum())
    assert abs(c.mean_accepted() - accepted.mean()) < 1e-12


# ----------------------------------------------------------------------------- the whole loop

@pytest.mark.parametrize("name,S,n,K,T,L,seed", [
    ("t_fp32", 3, 2, 3, 14, 5, 21),
    ("t_fp32", 1, 6, 1, 4, 4, 22),
    ("t_fp32", 5, 1, 2, 9, 5, 23),
])
def test_speculative_greedy_is_lossless(name, S, n, K, T, L, seed):
    cfg = ps.CONFIGS[name].replace(S=S, n=n)
    w = ps.make_weights(cfg, seed)
    prompt = ps.make_prompt(cfg, seed, 11)
    ref = po.plain_greedy(cfg, w, prompt, 24, NUM)
    out, ctr = po.speculative_greedy(cfg, w, prompt, 24, NUM, depth=L, topk=K, total=T)
    assert np.array_equal(ref, out)


@pytest.mark.parametrize("K,T,L,seed", [(3, 14, 5, 31), (1, 5, 5, 32), (2, 12, 5, 33)])
def test_lossless_with_multi_token_acceptance_and_compaction(K, T, L, seed):
    """A drafter that imitates the target makes rounds accept several tokens, so the commit path
    (cache compaction, several verified pairs entering the next round) is exercised; the stream
    must still be the plain greedy one and the compacted cache must equal a fresh prefill."""
    cfg = ps.CONFIGS["t_fp32"].replace(n_target_layers=1)
    w = ps.make_mimic_weights(cfg, seed)
    prompt = ps.make_prompt(cfg, seed, 9)
    ref = po.plain_greedy(cfg, w, prompt, 40, NUM)
    log = []
    out, ctr = po.speculative_greedy(cfg, w, prompt, 40, NUM, depth=L, topk=K, total=T, log=log)
    assert np.array_equal(ref, out)
    assert ctr.mean_accepted() > 1.0 and max(a for a, _ in log) >= 3
    assert ctr.rounds == len(log) and ctr.accepted_at[1] == sum(1 for a, _ in log if a >= 1)


def test_c1_lossless_128_tokens():
    cfg = ps.CONFIGS["c1"]
    w = ps.make_weights(cfg, 1)
    prompt = ps.make_prompt(cfg, 1, 64)
    ref = po.plain_greedy(cfg, w, prompt, 128, NUM)
    out, ctr = po.speculative_greedy(cfg, w, prompt, 128, NUM)
    assert np.array_equal(ref, out)


def test_commit_leaves_cache_equal_to_fresh_prefill():
    cfg = ps.CONFIGS["t_fp32"].replace(n_target_layers=1)
    w = ps.make_mimic_weights(cfg, 41)
    prompt = ps.make_prompt(cfg, 41, 9)
    n = len(prompt)
    kv = po.new_target_kv(cfg, 80, NUM)
    feat, logits = po.target_forward(cfg, w, kv, 0, prompt, np.arange(n), po.chain_parents(n), NUM)
    first = int(np.argmax(logits[-1]))
    dkv = np.zeros((cfg.S, 2, cfg.n_kv_heads, 80, cfg.head_dim))
    po.drafter_prefill(cfg, w, dkv, 0, prompt[1:], feat[:-1], NUM)
    tree = po.draft_round(cfg, w, dkv, n - 1, [first], feat[-1:], cfg.depth, cfg.topk, cfg.total, NUM)
    tf, tl = po.target_forward(cfg, w, kv, n, tree.tokens, n + tree.depth, tree.parents, NUM)
    path, a, bonus, nt, nf = po.verify_accept(tl, tf, tree.tokens, tree.parents)
    assert a >= 2
    for k in range(1, a + 1):
        kv[:, :, :, n + k, :] = kv[:, :, :, n + path[k], :]
    stream = np.concatenate([prompt, [first], nt[:-1]])
    kv2 = po.new_target_kv(cfg, 80, NUM)
    f2, _ = po.target_forward(cfg, w, kv2, 0, stream, np.arange(len(stream)), po.chain_parents(len(stream)), NUM)
    assert np.abs(kv[:, :, :, : len(stream)] - kv2[:, :, :, : len(stream)]).max() < 1e-9
    assert np.abs(nf - f2[n:]).max() < 1e-9           # features handed on are the target's own


# ----------------------------------------------------------------------------- a planted mistake is caught

def test_pins_catch_a_wrong_specialist_schedule(monkeypatch):
    """Sanity of the pins themselves: the typo'd subscript of Eq. 9 (ceil(i/n)) must fail the
    library-chain pin."""
    cfg = ps.CONFIGS["t_fp32"].replace(S=3, n=2, depth=5, topk=1, total=5)
    w = ps.make_weights(cfg, 5)
    toks, feats = ps.make_round_inputs(cfg, 5, n_new=4)
    want_tok, want_logp = drafter_chain_by_library(cfg, w, toks, feats, 5)
    monkeypatch.setattr(po, "specialist_for_position", lambda i, n, S: max(1, min(math.ceil(i / n), S)))
    res = po.draft_round(cfg, w, fresh_draft_kv(cfg, 5, 4, prefix=0), 0, toks, feats, 5, 1, 5, NUM)
    assert np.abs(res.scores[1:] - np.cumsum(want_logp)).max() > 1e-6


@pytest.mark.parametrize("mistake", ["dropped", "before_the_normalisation", "shifted", "none_means_unit_gain_norm"])
def test_pins_catch_a_wrong_rmsnorm_gain(monkeypatch, mistake):
    """The library pins must go red for a norm that drops its gain, applies it on the wrong side of the
    normalisation, reads it one column off, or treats an absent norm as a norm with gain 1."""
    def wrong(x, g, eps, num):
        x = np.asarray(x, dtype=num.dtype)
        if g is None:
            if mistake == "none_means_unit_gain_norm":
                return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)
            return x
        gw = num.w(g)
        if mistake == "dropped":
            return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)
        if mistake == "before_the_normalisation":
            y = x * gw
            return y / np.sqrt(np.mean(y * y, axis=-1, keepdims=True) + eps)
        if mistake == "shifted":
            return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps) * np.roll(gw, 1)
        return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps) * gw
    monkeypatch.setattr(po, "rmsnorm", wrong)
    if mistake == "none_means_unit_gain_norm":
        cfg = ps.CONFIGS["t_fp32"].replace(S=3, n=2, depth=5, topk=1, total=5, norm_in=False)
        w = ps.make_weights(cfg, 5)
        toks, feats = ps.make_round_inputs(cfg, 5, n_new=4)
        want_tok, want_logp = drafter_chain_by_library(cfg, w, toks, feats, 5)
        res = po.draft_round(cfg, w, fresh_draft_kv(cfg, 5, 4, prefix=0), 0, toks, feats, 5, 1, 5, NUM)
        assert np.abs(res.scores[1:] - np.cumsum(want_logp)).max() > 1e-4
        return
    cfg = ps.CONFIGS["t_fp32"]
    w = ps.make_weights(cfg, 2)
    m = hf_model(cfg, w, w["target"])
    prompt = ps.make_prompt(cfg, 2, 23)
    with torch.no_grad():
        out = m(torch.from_numpy(prompt.astype(np.int64))[None], output_hidden_states=True)
    kv = po.new_target_kv(cfg, 64, NUM)
    feat, logits = po.target_forward(cfg, w, kv, 0, prompt, np.arange(23), po.chain_parents(23), NUM)
    assert np.abs(out.logits[0].numpy() - logits).max() > 1e-3
    assert np.abs(out.hidden_states[-1][0].numpy() - feat).max() > 1e-3
