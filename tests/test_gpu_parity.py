"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded inputs."""
import math

import numpy as np
import pytest
import torch

import poss_synth as ps
from oracle import poss_oracle as po
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def make_poss(cfg, w, draft_slots, target_slots=0, **caps):
    from paper_2506_03566_b200 import Poss, make_config
    return Poss(make_config(cfg, draft_slots, target_slots, **caps), w)


def dev(a):
    from paper_2506_03566_b200 import to_device
    return to_device(a)


# ----------------------------------------------------------------------------- single stages

@pytest.mark.parametrize("name,M,N,K,impl", [
    ("t_fp32", 1, 777, 192, 1), ("t_fp32", 13, 344, 384, 1), ("t_fp32", 128, 8, 344, 1),
    ("t_bf16", 1, 512, 1024, 1), ("t_bf16", 57, 1408, 512, 1), ("t_bf16", 10, 5000, 512, 1),
])
def test_linear_matches_oracle(name, M, N, K, impl):
    cfg = ps.CONFIGS[name]
    w = ps.make_weights(cfg, 1)
    P = make_poss(cfg, w, 512)
    num = pu.oracle_num(cfg)
    x = ps.normal(3, "x", (M, K), 1.0, cfg.dtype)
    W = ps.normal(3, "w", (N, K), 0.02, cfg.dtype)
    b = ps.normal(3, "b", (N,), 0.02, cfg.dtype)
    res = ps.normal(3, "r", (M, N), 1.0, "fp32")
    got = P.poss_linear(dev(x), dev(W), dev(b), dev(res), impl=impl).cpu().numpy()
    want = po.linear(po.widen(x, num.dtype), W, num, b) + res
    assert np.abs(got - want).max() <= 1e-4
    got2 = P.poss_linear(dev(x), dev(W), impl=impl).cpu().numpy()
    assert np.abs(got2 - po.linear(po.widen(x, num.dtype), W, num)).max() <= 1e-4
    # M-invariance: a row's result does not depend on the batch it sits in
    if M > 1:
        one = P.poss_linear(dev(x[M - 1:M]), dev(W), impl=impl).cpu().numpy()
        assert np.array_equal(one[0], got2[M - 1])


@pytest.mark.parametrize("M,N,K", [
    (1, 128, 64), (10, 256, 512), (16, 5000, 512), (17, 777, 1024), (57, 4096, 1024), (64, 1408, 2048),
    (100, 384, 4096), (128, 130, 8192), (3, 640, 328),
])
def test_tensor_core_linear_matches_oracle_and_simt(M, N, K):
    """tcgen05 GEMM: several tiles, ragged N, K tails, split-K, every row-count padding."""
    cfg = ps.CONFIGS["t_bf16"]
    w = ps.make_weights(cfg, 1)
    P = make_poss(cfg, w, 512)
    num = pu.oracle_num(cfg)
    x = ps.normal(5, "x", (M, K), 1.0, "bf16")
    W = ps.normal(5, "w", (N, K), 0.02, "bf16")
    b = ps.normal(5, "b", (N,), 0.02, "bf16")
    res = ps.normal(5, "r", (M, N), 1.0, "fp32")
    got = P.poss_linear(dev(x), dev(W), dev(b), dev(res), impl=2).cpu().numpy()
    assert P.poss_last_status() == 0
    want = po.linear(po.widen(x, num.dtype), W, num, b) + res
    assert np.abs(got - want).max() <= 1e-4
    simt = P.poss_linear(dev(x), dev(W), dev(b), dev(res), impl=1).cpu().numpy()
    assert np.abs(got - simt).max() <= 1e-4
    # deterministic, and a row's value does not depend on the batch around it
    again = P.poss_linear(dev(x), dev(W), dev(b), dev(res), impl=2).cpu().numpy()
    assert np.array_equal(got, again)
    plain = P.poss_linear(dev(x), dev(W), impl=2).cpu().numpy()
    one = P.poss_linear(dev(x[M - 1:M]), dev(W), impl=2).cpu().numpy()
    assert np.array_equal(one[0], plain[M - 1])


@pytest.mark.parametrize("name,rows,P_len,Hq,Hkv,d", [
    ("t_fp32", 14, 37, 6, 2, 32), ("t_fp32", 1, 0, 4, 4, 64), ("t_fp32", 61, 300, 8, 1, 32),
    ("t_bf16", 25, 300, 8, 2, 64), ("t_bf16", 61, 1024, 32, 8, 128), ("t_bf16", 81, 2100, 8, 8, 128),
    ("t_bf16", 128, 5, 4, 1, 128),
])
def test_tree_attention_matches_oracle(name, rows, P_len, Hq, Hkv, d):
    cfg = ps.CONFIGS[name].replace(n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, hidden=Hq * d)
    w = ps.make_weights(cfg.replace(vocab=64, ffn=64), 1)
    P = make_poss(cfg.replace(vocab=64, ffn=64), w, 64)
    num = pu.oracle_num(cfg)
    cap = P_len + rows + 3
    q, kv = ps.make_attention_case(5, rows, Hq, Hkv, d, P_len, cap, cfg.dtype)
    parents = ps.random_tree_parents(6, rows)
    mask = po.pack_mask(po.ancestor_matrix(parents))
    scale = 1.0 / math.sqrt(d)
    got = pu.np_of(P.poss_tree_attention(dev(q), dev(kv), P_len, torch.from_numpy(mask.view(np.int64)).cuda(), scale))
    want = po.tree_attention(q, kv, P_len, parents, scale, num)
    pu.check_attention(got, want, cfg.dtype, f"tree {rows}x{P_len} Hq{Hq} Hkv{Hkv} d{d}")
    # chain mask = causal attention
    chain = po.pack_mask(po.ancestor_matrix(po.chain_parents(rows)))
    got_c = pu.np_of(P.poss_tree_attention(dev(q), dev(kv), P_len, torch.from_numpy(chain.view(np.int64)).cuda(), scale))
    want_c = po.tree_attention(q, kv, P_len, po.chain_parents(rows), scale, num)
    pu.check_attention(got_c, want_c, cfg.dtype, f"chain {rows}x{P_len} Hq{Hq} Hkv{Hkv} d{d}")


@pytest.mark.parametrize("rows,P_len,Hq,Hkv", [
    (1, 0, 8, 8), (16, 0, 8, 2), (5, 123, 8, 1), (5, 124, 8, 1), (61, 195, 16, 4), (61, 196, 16, 4),
    (128, 128, 4, 1), (128, 64, 8, 1), (40, 1987, 8, 2), (61, 1987, 8, 8), (61, 1988, 8, 2),
    (61, 4035, 8, 1), (10, 2100, 40, 40), (10, 8262, 32, 8), (10, 8262, 8, 1), (81, 8192, 8, 8), (128, 10112, 4, 4),
    (1, 10239, 8, 8), (70, 5000, 16, 2),
])
def test_tensor_core_tree_attention_at_its_block_boundaries(rows, P_len, Hq, Hkv):
    """Head dimension 128 (the tcgen05 kernel): key counts of 1 and 16, around the 128-key groups (128 / 129), the
    256-key units (256 / 257), 2048 / 2049 keys (where a (KV head, query tile) starts to be walked by CTAs that take
    several units each), 4096, the long-prefix draft and target shapes (8272 / 8273 keys: more than eight walkers, i.e.
    several clusters and the arrival counters) and the 10240-key limit; GQA groups of 1, 4 and 8; multi-head attention
    with 40 KV heads; one to eight query tiles; one and two mask words."""
    d = 128
    cfg = ps.CONFIGS["t_bf16"].replace(n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, hidden=Hq * d, vocab=64, ffn=64)
    P = make_poss(cfg, ps.make_weights(cfg, 1), 64)
    num = pu.oracle_num(cfg)
    cap = P_len + rows + 5
    q, kv = ps.make_attention_case(11, rows, Hq, Hkv, d, P_len, cap, cfg.dtype)
    scale = 1.0 / math.sqrt(d)
    for parents in (ps.random_tree_parents(12, rows), po.chain_parents(rows)):
        mask = po.pack_mask(po.ancestor_matrix(parents))
        got = pu.np_of(P.poss_tree_attention(dev(q), dev(kv), P_len, torch.from_numpy(mask.view(np.int64)).cuda(), scale))
        assert P.poss_last_status() == 0
        want = po.tree_attention(q, kv, P_len, parents, scale, num)
        pu.check_attention(got, want, "bf16", f"{rows}x{P_len} Hq{Hq} Hkv{Hkv}")


@pytest.mark.parametrize("rows,P_len,Hq,Hkv", [(10, 100, 8, 2), (61, 1024, 32, 8), (61, 1988, 8, 2), (10, 8262, 32, 8),
                                               (10, 2100, 40, 40)])
def test_the_tcgen05_attention_kernel_is_the_one_that_runs(rows, P_len, Hq, Hkv):
    """A launch the device refuses is handed to the split-KV kernels without an error; this checks, from the
    library's own launch records, that the tcgen05 kernel takes the shapes it is there for (one launch, no combine
    kernel), and that switching it off sends the same call to the mma.sync kernels."""
    from paper_2506_03566_b200.binding import POSS_OPT_ATTENTION_TCGEN05
    d = 128
    cfg = ps.CONFIGS["t_bf16"].replace(n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, hidden=Hq * d, vocab=64, ffn=64)
    P = make_poss(cfg, ps.make_weights(cfg, 1), 64)
    q, kv = ps.make_attention_case(11, rows, Hq, Hkv, d, P_len, P_len + rows, cfg.dtype)
    mask = torch.from_numpy(po.pack_mask(po.ancestor_matrix(po.chain_parents(rows))).view(np.int64)).cuda()
    qd, kvd = dev(q), dev(kv)
    P.poss_profile(3)
    a = P.poss_tree_attention(qd, kvd, P_len, mask, 1.0 / math.sqrt(d))
    names = [n for n, _ in P.poss_timeline_read()]
    assert names == ["attn_tc"], names
    P.poss_debug_option(POSS_OPT_ATTENTION_TCGEN05, 0)
    b = P.poss_tree_attention(qd, kvd, P_len, mask, 1.0 / math.sqrt(d))
    names = [n for n, _ in P.poss_timeline_read()]
    assert names[0] == "attn_mma" and "attn_tc" not in names, names
    P.poss_profile(0)
    assert P.poss_last_status() == 0
    # the two kernels group their sums differently: a bf16 unit apart at most
    assert (a.float() - b.float()).abs().max().item() <= 2e-2


def test_tensor_core_tree_attention_on_random_shapes():
    """24 seeded random shapes at head dimension 128 (1..64 rows, prefix 0..1500 and, every fourth trial, up to 9000;
    1..8 KV heads, GQA 1..8, cache capacity with and without slack, random trees and chains) against the oracle."""
    rng = np.random.default_rng(2024)
    d = 128
    ctxs = {}
    for trial in range(24):
        Hkv, G = int(rng.choice([1, 2, 4, 8])), int(rng.choice([1, 2, 4, 8]))
        Hq = Hkv * G
        rows = int(rng.integers(1, 65))
        P_len = int(rng.integers(0, 1501))
        if trial % 4 == 3:
            P_len = int(rng.integers(1500, 9001))
        cap = P_len + rows + int(rng.integers(0, 9))
        cfg = ps.CONFIGS["t_bf16"].replace(n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, hidden=Hq * d, vocab=64, ffn=64)
        if (Hq, Hkv) not in ctxs:
            ctxs[(Hq, Hkv)] = make_poss(cfg, ps.make_weights(cfg, 1), 64)
        P = ctxs[(Hq, Hkv)]
        q, kv = ps.make_attention_case(3000 + trial, rows, Hq, Hkv, d, P_len, cap, cfg.dtype)
        parents = ps.random_tree_parents(4000 + trial, rows) if trial % 3 else po.chain_parents(rows)
        mask = po.pack_mask(po.ancestor_matrix(parents))
        scale = 1.0 / math.sqrt(d)
        got = pu.np_of(P.poss_tree_attention(dev(q), dev(kv), P_len, torch.from_numpy(mask.view(np.int64)).cuda(), scale))
        assert P.poss_last_status() == 0
        want = po.tree_attention(q, kv, P_len, parents, scale, pu.oracle_num(cfg))
        pu.check_attention(got, want, "bf16", f"trial {trial}: {rows}x{P_len} Hq{Hq} Hkv{Hkv}")


def test_tree_root_row_equals_its_single_row_decode_bitwise():
    """The property the lossless loop rests on: a token whose visible keys are the prefix and itself gets the same
    attention output, bit for bit, as the root of a 61-row tree pass and as a single decoded row, also where the
    two calls cut their keys into different numbers of units and deal them to different numbers of CTAs (prefix 1000:
    1061 against 1001 keys; prefix 2040: 9 units on walkers that take two of them against 8 units)."""
    Hq, Hkv, d, rows = 32, 8, 128, 61
    cfg = ps.CONFIGS["t_bf16"].replace(n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, hidden=Hq * d, vocab=64, ffn=64)
    P = make_poss(cfg, ps.make_weights(cfg, 1), 64)
    scale = 1.0 / math.sqrt(d)
    tree = po.pack_mask(po.ancestor_matrix(ps.random_tree_parents(13, rows)))
    one = po.pack_mask(po.ancestor_matrix(po.chain_parents(1)))
    for P_len in (0, 100, 250, 1000, 1023, 1980, 2040, 4090, 8190):
        q, kv = ps.make_attention_case(14 + P_len, rows, Hq, Hkv, d, P_len, P_len + rows + 2, cfg.dtype)
        full = pu.np_of(P.poss_tree_attention(dev(q), dev(kv), P_len, torch.from_numpy(tree.view(np.int64)).cuda(), scale))
        single = pu.np_of(P.poss_tree_attention(dev(q[:1]), dev(kv), P_len, torch.from_numpy(one.view(np.int64)).cuda(), scale))
        assert P.poss_last_status() == 0
        assert np.array_equal(full[0], single[0]), f"root row differs at prefix {P_len}"


@pytest.mark.parametrize("name,rows,K", [("t_fp32", 3, 3), ("t_fp32", 1, 16), ("t_bf16", 4, 4), ("m_bf16", 10, 10),
                                         ("m_bf16", 61, 1), ("t_bf16", 128, 16), ("m_bf16", 64, 3), ("m_bf16", 17, 16)])
def test_lm_head_topk_matches_oracle(name, rows, K):
    cfg = ps.CONFIGS[name]
    w = ps.make_weights(cfg.replace(S=1, n_target_layers=0), 2)
    P = make_poss(cfg.replace(S=1, n_target_layers=0, topk=16, total=16, depth=2), w, 64)
    num = pu.oracle_num(cfg)
    f = ps.normal(4, "f", (rows, cfg.hidden), 1.5, cfg.dtype)
    ids, logp, logits = P.poss_lm_head_topk(dev(f), K, want_logits=True)
    ids, logp, logits = ids.cpu().numpy(), logp.cpu().numpy(), logits.cpu().numpy()
    z = po.linear(po.widen(f, num.dtype), w["lm_head"], num)
    tol = pu.TOL[cfg.dtype]
    assert np.abs(logits - z).max() <= tol
    lp = po.log_softmax_rows(z)
    want = po.topk_rows(z, K)
    for r in range(rows):
        if not np.array_equal(ids[r], want[r]):
            srt = np.sort(z[r])[::-1]
            assert po._decision_margin(srt, K) < pu.MARGIN, "top-k differs although the margin is large"
            assert np.all(z[r][ids[r]] >= srt[K - 1] - pu.MARGIN)
        assert np.abs(logp[r] - lp[r][ids[r]]).max() <= tol
    # the kernel's own logits decide its own top-k exactly (ties -> lowest id)
    own = po.topk_rows(logits.astype(np.float64), K)
    assert np.array_equal(own, ids)
    # the production form: lists built in the product's epilogue, the logits never stored (up to 16 rows: vocabulary
    # rows on the accumulator's lanes and warp-wide lists; more rows: one thread per activation row)
    ids2, logp2, _ = P.poss_lm_head_topk(dev(f), K)
    ids2, logp2 = ids2.cpu().numpy(), logp2.cpu().numpy()
    assert P.poss_last_status() == 0
    for r in range(rows):
        if not np.array_equal(ids2[r], want[r]):
            srt = np.sort(z[r])[::-1]
            assert po._decision_margin(srt, K) < pu.MARGIN, "fused top-k differs although the margin is large"
            assert np.all(z[r][ids2[r]] >= srt[K - 1] - pu.MARGIN)
        assert len(set(ids2[r].tolist())) == K
        assert np.abs(logp2[r] - lp[r][ids2[r]]).max() <= tol


def test_lm_head_topk_exact_ties_go_to_the_lowest_id():
    cfg = ps.CONFIGS["t_fp32"].replace(S=1, n_target_layers=0)
    w = ps.make_weights(cfg, 2)
    w["lm_head"][5] = w["lm_head"][700]
    w["lm_head"][300] = w["lm_head"][700]
    P = make_poss(cfg, w, 64)
    f = (w["lm_head"][700:701] * 400).astype(np.float32)        # rows 5, 300, 700 tie for the maximum
    ids, logp, _ = P.poss_lm_head_topk(dev(f), 3)
    assert ids.cpu().numpy().tolist() == [[5, 300, 700]]
    assert logp[0, 0] == logp[0, 1] == logp[0, 2]


def test_verify_accept_planted_paths():
    cfg = ps.CONFIGS["t_bf16"].replace(S=1, n_target_layers=0, vocab=5000)
    w = ps.make_weights(cfg, 3)
    P = make_poss(cfg, w, 64)
    rows = 61
    parents = ps.random_tree_parents(8, rows, max_children=4)
    g = np.random.default_rng(0)
    tokens = np.zeros(rows, dtype=np.int32)
    for p in range(rows):
        kids = [c for c in range(rows) if parents[c] == p]
        tokens[kids] = g.permutation(cfg.vocab)[: len(kids)]
    anc = po.ancestor_matrix(parents)
    feats = ps.normal(9, "tf", (rows, cfg.hidden), 1.0, "bf16")
    P.poss_reset()
    accepted = []
    for target_node in [0, 17, 60, int(np.argmax(anc.sum(1)))]:
        path = [j for j in range(rows) if anc[target_node, j]]
        logits = ps.normal(10 + target_node, "lg", (rows, cfg.vocab), 1.0, "bf16")
        lg = po.widen(logits, np.float32).copy()
        for a_, b_ in zip(path[:-1], path[1:]):
            lg[a_, tokens[b_]] += 12.0
        # make sure the walk stops at target_node: its argmax must not be a child token
        kids = [int(tokens[c]) for c in range(rows) if parents[c] == target_node]
        lg[target_node, kids] -= 30.0
        lg_bits = ps._to_bf16_bits(lg.astype(np.float32).ravel()).reshape(rows, cfg.vocab)
        lg = po.widen(lg_bits, np.float64)
        want = po.verify_accept(lg, po.widen(feats, np.float64), tokens, parents)
        out = P.poss_verify_accept(dev(lg_bits), None, dev(feats), torch.from_numpy(tokens).cuda(),
                                   torch.from_numpy(parents).cuda(), rows)
        a = int(out["n_accepted"][0])
        assert a == want[1] == len(path) - 1
        assert out["path"][: a + 1].cpu().tolist() == want[0]
        assert int(out["bonus"][0]) == want[2]
        assert out["new_tokens"][: a + 1].cpu().tolist() == want[3].tolist()
        assert np.array_equal(pu.np_of(out["new_features"][: a + 1]), want[4])
        # same through the argmax entry
        gmax = torch.from_numpy(po.argmax_rows(lg)).cuda()
        out2 = P.poss_verify_accept(None, gmax, dev(feats), torch.from_numpy(tokens).cuda(),
                                    torch.from_numpy(parents).cuda(), rows)
        assert out2["path"].cpu().tolist() == out["path"].cpu().tolist()
        accepted += [a, a]
    rounds, n_at = P.poss_get_counters()
    ctr = po.Counters(cfg.depth)
    for a in accepted:
        ctr.add(min(a, cfg.depth))
    assert rounds == len(accepted)
    for i in range(1, cfg.depth + 1):
        assert n_at[i] == sum(1 for a in accepted if a >= i)


@pytest.mark.parametrize("name,vocab,rows,temperature", [
    ("t_fp32", 777, 14, 1.0), ("t_bf16", 5000, 25, 1.0), ("t_bf16", 5000, 61, 0.7), ("t_bf16", 33, 61, 1.0),
    ("t_bf16", 32003, 128, 1.0), ("t_bf16", 5000, 1, 1.0),
])
def test_verify_sample_matches_oracle(name, vocab, rows, temperature):
    """Verification at a temperature: the walk, the bonus token, the verified pairs and the number of uniforms used
    equal the oracle's for 24 different uniform streams per case (decisions compare a uniform with a probability:
    fp32 on the GPU, fp64 in the oracle, so a uniform within 1e-5 of its threshold could legitimately flip; with
    these seeds none is).  Child tokens get a boost so that walks of every depth occur."""
    cfg = ps.CONFIGS[name].replace(S=1, n_target_layers=0, vocab=vocab)
    P = make_poss(cfg, ps.make_weights(cfg, 3), 64)
    parents = ps.random_tree_parents(40 + rows, rows, max_children=4)
    g = np.random.default_rng(rows)
    tokens = np.zeros(rows, dtype=np.int32)
    for p in range(rows):
        kids = [c for c in range(rows) if parents[c] == p]
        tokens[kids] = g.permutation(vocab)[: len(kids)]
    logits = (g.standard_normal((rows, vocab)) * 2.0).astype(np.float32)
    for c in range(1, rows):
        logits[parents[c], tokens[c]] += 5.0
    feats = ps.normal(9, "tf", (rows, cfg.hidden), 1.0, cfg.dtype)
    feats_wide = po.widen(feats, np.float64)
    lg_d, feats_d = torch.from_numpy(logits).cuda(), dev(feats)
    tok_d, par_d = torch.from_numpy(tokens).cuda(), torch.from_numpy(parents).cuda()
    P.poss_reset()
    depths = []
    for trial in range(24):
        u = np.random.default_rng(1000 * rows + trial).random(max(rows, 2)).astype(np.float32)
        if trial == 0:
            u[:] = 0.0                        # accepts every first child down to a leaf
        if trial == 1:
            u[:] = np.float32(1.0 - 2.0 ** -24)   # rejects everything: the bonus comes from the root's residual
        path, a, bonus, used = po.sample_walk(logits, tokens, parents, temperature, u)
        out = P.poss_verify_sample(lg_d, feats_d, tok_d, par_d, rows, temperature, torch.from_numpy(u).cuda())
        assert P.poss_last_status() == 0
        a_cap = min(a, 16)
        assert int(out["n_accepted"][0]) == a == a_cap, f"trial {trial}"
        assert out["path"][: a + 1].cpu().tolist() == path
        assert int(out["bonus"][0]) == bonus, f"trial {trial}"
        assert int(out["uniforms_used"][0]) == used
        want_tokens = [int(tokens[j]) for j in path[1:]] + [bonus]
        assert out["new_tokens"][: a + 1].cpu().tolist() == want_tokens
        assert np.array_equal(pu.np_of(out["new_features"][: a + 1]), feats_wide[path])
        depths.append(a)
    if rows > 1:
        assert max(depths) >= 2 and min(depths) == 0
    rounds, n_at = P.poss_get_counters()
    assert rounds == 24
    for i in range(1, cfg.depth + 1):
        assert n_at[i] == sum(1 for a in depths if a >= i)


def test_verify_sample_argument_errors():
    cfg = ps.CONFIGS["t_bf16"].replace(S=1, n_target_layers=0)
    P = make_poss(cfg, ps.make_weights(cfg, 3), 64)
    rows = 5
    lg = torch.zeros((rows, cfg.vocab), dtype=torch.float32, device="cuda")
    feats = torch.zeros((rows, cfg.hidden), dtype=torch.bfloat16, device="cuda")
    tok = torch.zeros(rows, dtype=torch.int32, device="cuda")
    par = torch.tensor([-1, 0, 0, 1, 1], dtype=torch.int32, device="cuda")
    few = torch.zeros(rows - 1, dtype=torch.float32, device="cuda")
    with pytest.raises(Exception):
        P.poss_verify_sample(lg, feats, tok, par, rows, 1.0, few)          # fewer uniforms than rows
    with pytest.raises(Exception):
        P.poss_verify_sample(lg, feats, tok, par, rows, 0.0, torch.zeros(rows, dtype=torch.float32, device="cuda"))


# ----------------------------------------------------------------------------- the draft round

ROUND_CASES = [
    # name, overrides, n_new, seed, require_exact
    ("c1", {}, 1, 1, True),
    ("c1", {}, 5, 2, True),
    ("t_fp32", {}, 1, 3, True),
    ("t_fp32", {}, 4, 4, True),
    ("t_fp32", {"S": 1, "n": 5}, 2, 5, True),
    ("t_fp32", {"S": 5, "n": 1, "topk": 4, "total": 30}, 3, 6, True),
    ("t_fp32", {"depth": 1, "topk": 1, "total": 1}, 7, 7, True),
    ("t_fp32", {"depth": 2, "topk": 2, "total": 3}, 1, 8, True),       # round shallower than the schedule
    ("t_bf16", {}, 1, 9, False),
    ("t_bf16", {}, 6, 10, False),
    ("t_bf16", {"S": 6, "n": 1, "topk": 10, "total": 60}, 2, 11, False),
    ("m_bf16", {}, 1, 12, False),
    ("m_bf16", {"S": 3, "n": 2}, 7, 13, False),
    ("m_bf16", {"S": 4, "n": 2, "depth": 8, "total": 80}, 3, 14, False),
    # the kernels' limits: 128 rows in one projection batch (8 verified pairs + 120 tree slots = (depth-1)*topk),
    # 255 kept tokens (four mask words per row), 1815 candidates in the rerank; width 16 at depth 8
    # (cumulative scores near -50 at depth 9: an fp32 unit there is 4e-6, so two candidates 1e-6 apart in the fp64
    # oracle may swap places on the GPU; the teacher-forced comparison with the margin rule covers that)
    ("t_fp32", {"S": 3, "n": 3, "depth": 9, "topk": 15, "total": 255}, 1, 15, False),
    ("t_bf16", {"S": 2, "n": 5, "depth": 9, "topk": 15, "total": 200}, 8, 16, False),
    ("t_bf16", {"S": 4, "n": 2, "depth": 8, "topk": 16, "total": 100}, 3, 19, False),
    # degenerate: one step, one candidate; chain drafting in bf16
    ("t_bf16", {"depth": 1, "topk": 1, "total": 1}, 1, 17, False),
    ("t_bf16", {"S": 6, "n": 1, "depth": 6, "topk": 1, "total": 6}, 2, 18, False),
    # draft layers without an input norm (norm_in = NULL: the attention reads fc's output as it is)
    ("t_fp32", {"norm_in": False}, 3, 24, True),
    ("t_bf16", {"norm_in": False}, 2, 25, False),
    # rows wider than 8192 columns: the norm kernel's loop over the column groups it does not keep in registers
    ("t_bf16", {"hidden": 8448, "S": 2, "n": 1, "depth": 2, "topk": 2, "total": 4, "vocab": 777, "ffn": 344}, 2, 26, False),
    ("t_fp32", {"hidden": 8264, "S": 1, "n": 2, "depth": 2, "topk": 2, "total": 4, "vocab": 333, "ffn": 120}, 2, 27, True),
]


@pytest.mark.parametrize("name,over,n_new,seed,require_exact", ROUND_CASES)
def test_draft_round_matches_oracle(name, over, n_new, seed, require_exact):
    cfg = ps.CONFIGS[name].replace(n_target_layers=0, **over)
    w = ps.make_weights(cfg, seed)
    cap = cfg.prefix + n_new + cfg.tree_slots
    P = make_poss(cfg, w, cap)
    kv = ps.make_draft_kv(cfg, seed, cap)
    tok, feat = ps.make_round_inputs(cfg, seed, n_new)
    g, trace, dkv = pu.run_gpu_round(P, cfg, kv, cfg.prefix, tok, feat, cfg.depth, cfg.topk, cfg.total)
    num = pu.oracle_num(cfg)
    rep = pu.compare_round(cfg, w, kv, cfg.prefix, tok, feat, cfg.depth, cfg.topk, cfg.total, g, trace, num,
                           require_exact)
    # verified pairs are cached by every specialist, in cache precision
    pu.compare_kv(cfg, dkv, rep["kv_oracle"], cfg.prefix, cfg.prefix + n_new, pu.TOL[cfg.dtype])
    print(name, over, {k: v for k, v in rep.items() if k != "kv_oracle"})
    # run-to-run bit equality (ordered reductions; no atomics on values)
    g2, trace2, _ = pu.run_gpu_round(P, cfg, kv, cfg.prefix, tok, feat, cfg.depth, cfg.topk, cfg.total)
    for k in ("tokens", "parents", "scores", "depth", "anc_mask"):
        assert np.array_equal(g[k], g2[k])
    assert np.array_equal(trace["step_features"], trace2["step_features"])


@pytest.mark.parametrize("name,over,B,seed", [
    ("t_fp32", {}, 3, 61),                                   # check mode, 3 specialists x 2 positions
    ("t_bf16", {}, 7, 62),                                   # the row limit: 7 sequences' pending + current rows
    ("t_bf16", {"S": 1, "n": 6, "norm_in": False}, 16, 63),  # the batch limit, one specialist, no input norm
    ("m_bf16", {}, 2, 64),                                   # six specialists, width 10: two sequences fit
    ("m_bf16", {"S": 1, "n": 6}, 12, 65),                    # one specialist, width 10: twelve sequences (120 rows)
    ("t_bf16", {"head_dim": 128, "n_q_heads": 4, "n_kv_heads": 2, "S": 2, "n": 3}, 5, 66),   # tcgen05 attention
])
def test_batched_draft_round_equals_single_rounds_bitwise_and_the_oracle(name, over, B, seed):
    """poss_draft_round_batched: sequences with different prefix lengths, different numbers of verified pairs, their
    own caches and inputs.  Every sequence's tree, scores, per-step features and cache entries equal, bit for bit,
    what poss_draft_round gives for that sequence alone (the products see more rows, and a row's value does not
    depend on the rows around it), and each sequence matches the oracle's definition -- independent rounds -- under
    the rules of the single-sequence test."""
    cfg = ps.CONFIGS[name].replace(n_target_layers=0, **over)
    w = ps.make_weights(cfg, seed)
    n_news = [1 + (b % 3) for b in range(B)]
    prefixes = [cfg.prefix - 5 * b for b in range(B)]
    cap = cfg.prefix + 3 + cfg.tree_slots
    from paper_2506_03566_b200 import Poss, make_config
    P = Poss(make_config(cfg, cap, 0, max_batch=B), w)
    kvs_np = [ps.make_draft_kv(cfg, seed + 100 * b, cap, prefixes[b]) for b in range(B)]
    ins = [ps.make_round_inputs(cfg, seed + 100 * b, n_news[b]) for b in range(B)]
    tok_all = torch.from_numpy(np.concatenate([t for t, _ in ins])).cuda()
    feat_all = dev(np.concatenate([f for _, f in ins], axis=0))
    kvs = [dev(k) for k in kvs_np]
    out = P.poss_draft_round_batched(kvs, prefixes, tok_all, feat_all, n_news, cfg.depth, cfg.topk, cfg.total)
    torch.cuda.synchronize()
    assert P.poss_last_status() == 0
    host = {k: pu.np_of(v) for k, v in out.items()}
    traces = [{k: pu.np_of(v) for k, v in P.poss_draft_trace(cfg.depth, cfg.topk, int(host["n_nodes"][b]), seq=b).items()}
              for b in range(B)]
    num = pu.oracle_num(cfg)
    for b in range(B):
        g1, tr1, dkv1 = pu.run_gpu_round(P, cfg, kvs_np[b], prefixes[b], ins[b][0], ins[b][1], cfg.depth, cfg.topk, cfg.total)
        gb = {k: (host[k][b] if k != "n_nodes" else host[k][b:b + 1]) for k in host}
        gb["anc_mask"] = gb["anc_mask"].view(np.uint64)
        for k in ("tokens", "parents", "scores", "depth", "anc_mask", "n_nodes"):
            assert np.array_equal(gb[k], g1[k]), (b, k)
        for k in tr1:
            assert np.array_equal(traces[b][k], tr1[k]), (b, k)
        assert torch.equal(kvs[b], dkv1), f"sequence {b}: cache entries differ from the single round's"
        if b in (0, B - 1):                                  # the oracle comparison proper, on the batch's two ends
            rep = pu.compare_round(cfg, w, kvs_np[b], prefixes[b], ins[b][0], ins[b][1], cfg.depth, cfg.topk, cfg.total,
                                   gb, traces[b], num, cfg.dtype == "fp32")
            pu.compare_kv(cfg, kvs[b], rep["kv_oracle"], prefixes[b], prefixes[b] + n_news[b],
                          pu.TOL[cfg.dtype])


def test_batched_round_capacity_errors():
    from paper_2506_03566_b200 import Poss, PossError, make_config
    cfg = ps.CONFIGS["t_bf16"].replace(n_target_layers=0)
    cap = cfg.prefix + 3 + cfg.tree_slots
    P = Poss(make_config(cfg, cap, 0, max_batch=8), ps.make_weights(cfg, 1))
    kv = [P.new_draft_kv() for _ in range(9)]
    tok = torch.zeros(9, dtype=torch.int32, device="cuda")
    feat = torch.zeros((9, cfg.hidden), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(PossError) as e:                      # more sequences than the context was sized for
        P.poss_draft_round_batched(kv, [10] * 9, tok, feat, [1] * 9, cfg.depth, cfg.topk, cfg.total)
    assert e.value.code == 3
    with pytest.raises(PossError) as e:                      # 8 x (1 + 3 x 4 + 4) + ... rows exceed one product
        P.poss_draft_round_batched(kv[:8], [10] * 8, tok[:8], feat[:8], [1] * 8, cfg.depth, cfg.topk, cfg.total)
    assert e.value.code == 3
    with pytest.raises(PossError) as e:
        P.poss_draft_round_batched(kv[:2], [10, -1], tok[:2], feat[:2], [1, 1], cfg.depth, cfg.topk, cfg.total)
    assert e.value.code == 1
    assert P.poss_last_status() == 0


def test_alternative_kernel_paths_give_the_same_round_bitwise():
    """Two kernels exist for two stages and the library picks one per call; the choice must not show in the
    result.  The gate/up product finished by the GEMM's own SwiGLU epilogue (POSS_OPT_SWIGLU_IN_KERNEL) against the
    consumer kernel over the parked partials: both add a tile's partials in range order and apply the same SiLU,
    so a whole draft round is equal bit for bit wherever both cut the product into the same CTA ranges, i.e. with
    more tiles than half the grid (ffn 4864 = 76 tiles here, 224 at full size; with fewer tiles the parked-partials
    path trims its grid to a multiple of the tile count and the two agree to rounding only).  (The two attention
    kernels group their sums differently and agree to a bf16 unit: they are compared with the oracle in the
    attention tests.)"""
    cfg = ps.CONFIGS["m_bf16"].replace(ffn=4864)
    w = ps.make_weights(cfg, 12)
    cap = cfg.prefix + 8 + cfg.tree_slots
    tok, feat = ps.make_round_inputs(cfg, 12, 3)
    outs = []
    from paper_2506_03566_b200.binding import POSS_OPT_SWIGLU_IN_KERNEL
    for flag in (0, 1):
        P = make_poss(cfg, w, cap)
        P.poss_debug_option(POSS_OPT_SWIGLU_IN_KERNEL, flag)
        dkv = dev(ps.make_draft_kv(cfg, 12, cap))
        out = P.poss_draft_round(dkv, cfg.prefix, torch.from_numpy(tok).cuda(), dev(feat), cfg.depth, cfg.topk, cfg.total)
        assert P.poss_last_status() == 0
        outs.append({k: v.cpu().numpy().copy() for k, v in out.items()} | {"kv": pu.np_of(dkv)})
    for k in outs[0]:
        assert np.array_equal(outs[0][k], outs[1][k]), k


def test_aliased_specialists_equal_single_layer_bitwise():
    base = ps.CONFIGS["t_bf16"]
    tok, feat = ps.make_round_inputs(base, 21, 3)
    ref = None
    for S, n in [(1, 6), (3, 2), (6, 1)]:
        cfg = base.replace(S=S, n=n, n_target_layers=0)
        w = ps.make_weights(cfg, 21, alias_specialists=True)
        cap = cfg.prefix + 3 + cfg.tree_slots
        kv = ps.make_draft_kv(cfg.replace(S=1), 21, cap)
        kv = np.repeat(kv, S, axis=0)
        P = make_poss(cfg, w, cap)
        g, trace, _ = pu.run_gpu_round(P, cfg, kv, cfg.prefix, tok, feat, cfg.depth, cfg.topk, cfg.total)
        if ref is None:
            ref = (g, trace)
        else:
            for k in ("tokens", "parents", "scores", "depth"):
                assert np.array_equal(g[k], ref[0][k]), k
            assert np.array_equal(trace["step_features"], ref[1]["step_features"])


def test_draft_prefill_matches_oracle_and_round_from_prefix():
    cfg = ps.CONFIGS["t_bf16"].replace(n_target_layers=0)
    w = ps.make_weights(cfg, 22)
    n = 150                                  # more than one chunk of POSS_MAX_ROWS
    cap = n + 8 + cfg.tree_slots
    P = make_poss(cfg, w, cap)
    toks = ps.tokens(22, "pf", n, cfg.vocab)
    feats = ps.normal(22, "pff", (n, cfg.hidden), 1.0, cfg.dtype)
    dkv = P.new_draft_kv()
    P.poss_draft_prefill(dkv, 0, torch.from_numpy(toks).cuda(), dev(feats))
    num = pu.oracle_num(cfg)
    kv_o = np.zeros((cfg.S, 2, cfg.n_kv_heads, cap, cfg.head_dim))
    po.drafter_prefill(cfg, w, kv_o, 0, toks, feats, num)
    pu.compare_kv(cfg, dkv, kv_o, 0, n, 2e-2)


def test_capacity_and_argument_errors_are_reported():
    from paper_2506_03566_b200 import PossError
    cfg = ps.CONFIGS["t_fp32"].replace(n_target_layers=0)
    w = ps.make_weights(cfg, 1)
    P = make_poss(cfg, w, 64)
    kv = P.new_draft_kv()
    tok = torch.zeros(1, dtype=torch.int32, device="cuda")
    feat = torch.zeros((1, cfg.hidden), device="cuda")
    for args, code in [((kv, 60, tok, feat, cfg.depth, cfg.topk, cfg.total), 3),      # cache too small
                       ((kv, 0, tok, feat, cfg.depth + 1, cfg.topk, cfg.total), 3),   # depth over the capacity
                       ((kv, 0, tok, feat, cfg.depth, cfg.topk + 1, cfg.total), 3),
                       ((kv, -1, tok, feat, cfg.depth, cfg.topk, cfg.total), 1)]:
        with pytest.raises(PossError) as e:
            P.poss_draft_round(*args)
        assert e.value.code == code
    assert P.poss_last_status() == 0


# ----------------------------------------------------------------------------- target pass and the full loop

@pytest.mark.parametrize("name,n,rows", [("t_fp32", 40, 25), ("t_bf16", 40, 25), ("t_bf16", 130, 64), ("t_bf16", 7, 128)])
def test_target_forward_tree_rows_match_oracle(name, n, rows):
    """Prefill (one or two chunks) and a tree pass; 64 rows is the widest argmax-epilogue launch, 128 the row limit."""
    cfg = ps.CONFIGS[name]
    w = ps.make_weights(cfg, 31)
    P = make_poss(cfg, w, 64, n + rows + 8)
    num = pu.oracle_num(cfg)
    prompt = ps.make_prompt(cfg, 31, n)
    tkv = P.new_target_kv()
    feats, arg = P.poss_target_prefill(tkv, 0, torch.from_numpy(prompt).cuda())
    kv_o = po.new_target_kv(cfg, n + rows + 8, num)
    f_o, l_o = po.target_forward(cfg, w, kv_o, 0, prompt, np.arange(n), po.chain_parents(n), num)
    tol = pu.TOL[cfg.dtype]
    assert np.abs(pu.np_of(feats) - f_o).max() <= tol
    parents = ps.random_tree_parents(32, rows)
    depth = np.zeros(rows, dtype=np.int32)
    for r in range(1, rows):
        depth[r] = depth[parents[r]] + 1
    toks = ps.tokens(33, "tt", rows, cfg.vocab)
    mask = po.pack_mask(po.ancestor_matrix(parents))
    tf, targ, tl = P.poss_target_forward(tkv, n, torch.from_numpy(toks).cuda(), torch.from_numpy(depth).cuda(),
                                         torch.from_numpy(mask.view(np.int64)).cuda(), rows, want_logits=True)
    f2, l2 = po.target_forward(cfg, w, kv_o, n, toks, n + depth, parents, num)
    assert np.abs(pu.np_of(tf) - f2).max() <= tol
    assert np.abs(tl.cpu().numpy() - l2).max() <= tol
    want_arg = po.argmax_rows(l2)
    got_arg = targ.cpu().numpy()
    for r in range(rows):
        if got_arg[r] != want_arg[r]:
            srt = np.sort(l2[r])[::-1]
            assert srt[0] - srt[1] < pu.MARGIN


def _loop_case(cfg, w, seed, n_prompt, n_gen, depth, topk, total):
    from paper_2506_03566_b200 import speculative_generate, plain_generate
    slots = n_prompt + n_gen + total + depth + 4
    P = make_poss(cfg, w, slots + (depth - 1) * topk, slots, max_depth=depth, max_topk=topk, max_total=total)
    prompt = ps.make_prompt(cfg, seed, n_prompt)
    pt = torch.from_numpy(prompt).cuda()
    log = []
    spec = speculative_generate(P, pt, n_gen, depth, topk, total, log=log)
    plain = plain_generate(P, pt, n_gen)
    assert P.poss_last_status() == 0
    return P, prompt, spec, plain, log


def test_c1_full_loop_is_lossless_and_equals_the_oracle_stream():
    cfg = ps.CONFIGS["c1"]
    w = ps.make_weights(cfg, 1)
    P, prompt, spec, plain, log = _loop_case(cfg, w, 1, 64, 128, cfg.depth, cfg.topk, cfg.total)
    want = po.plain_greedy(cfg, w, prompt, 128, po.Num())
    assert spec == plain == want.tolist()


@pytest.mark.parametrize("K,T,L,seed", [(3, 14, 5, 31), (1, 5, 5, 32), (2, 12, 5, 33)])
def test_loop_with_multi_token_acceptance_is_lossless(K, T, L, seed):
    cfg = ps.CONFIGS["t_fp32"].replace(n_target_layers=1)
    w = ps.make_mimic_weights(cfg, seed)
    P, prompt, spec, plain, log = _loop_case(cfg, w, seed, 9, 40, L, K, T)
    want = po.plain_greedy(cfg, w, prompt, 40, po.Num())
    olog = []
    ospec, octr = po.speculative_greedy(cfg, w, prompt, 40, po.Num(), depth=L, topk=K, total=T, log=olog)
    assert spec == plain == want.tolist()
    assert [a for a, _ in log] == [a for a, _ in olog]          # same accepted lengths, round by round
    assert [p for _, p in log] == [p for _, p in olog]          # same accepted paths
    rounds, n_at = P.poss_get_counters()
    assert rounds == octr.rounds and n_at[1:L + 1] == octr.accepted_at[1:L + 1].tolist()
    assert max(a for a, _ in log) >= 3


def test_sampling_loop_at_a_vanishing_temperature_is_the_greedy_loop():
    """The loop with poss_verify_sample at temperature 1e-4 (every target distribution a point mass on its argmax)
    emits the greedy stream with the greedy loop's accepted paths, whatever the uniforms; at temperature 1 it runs,
    accepts draft tokens, and two runs from the same generator seed agree."""
    from paper_2506_03566_b200 import speculative_generate
    cfg = ps.CONFIGS["t_fp32"].replace(n_target_layers=1)
    w = ps.make_mimic_weights(cfg, 31)
    P, prompt, spec, plain, log = _loop_case(cfg, w, 31, 9, 40, 5, 3, 14)
    pt = torch.from_numpy(prompt).cuda()
    gen = torch.Generator(device="cuda").manual_seed(5)
    slog = []
    cold = speculative_generate(P, pt, 40, 5, 3, 14, log=slog, temperature=1e-4, generator=gen)
    assert P.poss_last_status() == 0
    assert cold == spec and slog == log
    runs = []
    for _ in range(2):
        gen.manual_seed(6)
        hlog = []
        runs.append((speculative_generate(P, pt, 40, 5, 3, 14, log=hlog, temperature=1.0, generator=gen), hlog))
    assert P.poss_last_status() == 0
    assert runs[0] == runs[1] and len(runs[0][0]) == 40
    assert all(0 <= t < cfg.vocab for t in runs[0][0])


def test_bf16_loop_is_lossless_against_its_own_plain_decode():
    cfg = ps.CONFIGS["t_bf16"].replace(n_target_layers=1)
    w = ps.make_mimic_weights(cfg, 41)
    P, prompt, spec, plain, log = _loop_case(cfg, w, 41, 17, 48, 5, 3, 14)
    # bf16: tree rows and single rows go through the same reduction orders, so the streams agree;
    # a difference must be explained by a near-tie in the oracle's logits at that position
    if spec != plain:
        i = next(k for k in range(len(spec)) if spec[k] != plain[k])
        num = pu.oracle_num(cfg)
        stream = np.concatenate([prompt, np.array(plain[:i], dtype=np.int32)])
        kv_o = po.new_target_kv(cfg, len(stream) + 1, num)
        _, lg = po.target_forward(cfg, w, kv_o, 0, stream, np.arange(len(stream)), po.chain_parents(len(stream)), num)
        srt = np.sort(lg[-1])[::-1]
        assert srt[0] - srt[1] < pu.MARGIN, "streams diverge without a near-tie"
    assert sum(a for a, _ in log) > 0


def test_round_on_a_side_stream_equals_the_default_stream_bitwise():
    """All work is enqueued on the caller's stream: the same round on a non-default stream, with other work
    running on the default stream meanwhile, gives the same bits."""
    cfg = ps.CONFIGS["t_bf16"].replace(n_target_layers=0)
    w = ps.make_weights(cfg, 51)
    cap = cfg.prefix + 2 + cfg.tree_slots
    P = make_poss(cfg, w, cap)
    kv = ps.make_draft_kv(cfg, 51, cap)
    tok, feat = ps.make_round_inputs(cfg, 51, 2)
    g, trace, _ = pu.run_gpu_round(P, cfg, kv, cfg.prefix, tok, feat, cfg.depth, cfg.topk, cfg.total)
    side = torch.cuda.Stream()
    noise = torch.randn(4096, 4096, device="cuda")
    with torch.cuda.stream(side):
        for _ in range(3):
            noise_out = noise @ noise                    # unrelated work on the default stream's neighbour
        g2, trace2, _ = pu.run_gpu_round(P, cfg, kv, cfg.prefix, tok, feat, cfg.depth, cfg.topk, cfg.total)
    torch.cuda.synchronize()
    for k in ("tokens", "parents", "scores", "depth", "anc_mask"):
        assert np.array_equal(g[k], g2[k]), k
    assert np.array_equal(trace["step_features"], trace2["step_features"])
    assert P.poss_last_status() == 0
