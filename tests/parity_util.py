"""Shared helpers of the GPU parity tests: run a draft round through the C library, run the oracle on
the same seeded inputs, and compare under the stated rules.

Rules (written here, used by every parity test):
  * check mode (fp32): structure, tokens and paths bit-exact; features/logits within 1e-4.
  * bf16: features/logits/log-probs within 2e-2.  Where a full-size test hands in a second oracle precision
    (`noise_num`), the distance between the two oracles on the same step (both correct, both under the same bf16
    contract, fp32 against fp64 arithmetic between the rounding points) is measured and the feature bound is
    max(2e-2, 3 x that distance), never more than 2e-2 x max(1, RMS of the step's features): two correct bf16
    implementations differ by whole bf16 units wherever a rounding flips, and that floor depends on the shape.
    Structure bit-exact unless the oracle's margin at the
    deciding comparison is below 1e-2.  bf16 results of two correct implementations agree only to
    about one bf16 unit per rounding boundary, and that noise grows with the draft depth, so the
    numeric comparison is PER STEP WITH TEACHER FORCING: the oracle is re-run following the GPU's
    decisions and taking the GPU's previous-step features and parent scores as inputs (all arithmetic
    of the step is the oracle's own).  The step's two stages are compared separately: the feature against
    the oracle's feature from the previous step's inputs, the LM head / log-softmax / top-k against the
    oracle's head applied to the GPU's feature of the same step.  Every GPU decision must be valid up to the margin under the
    oracle's values; decisions that differ from the oracle's own choice are counted and reported.
"""
from __future__ import annotations

import numpy as np
import torch

import poss_synth as ps
from oracle import poss_oracle as po

MARGIN = 1e-2
TOL = {"fp32": 1e-4, "bf16": 2e-2}


# Tree attention output in bf16: the result is rounded to bf16 once (half a unit = 2^-9 of the element), the softmax
# and both products carry fp32-level error (the probabilities enter P.V with 16 significant bits).  The bound is per
# element: one whole bf16 unit of the element plus a floor relative to the output's RMS (the outputs of N(0,1) values
# averaged over n keys have RMS ~ sqrt(e/n), e.g. 0.04 at 2000 keys: an absolute bound would not bite there).
ATTN_FLOOR_REL = {"bf16": 2.0e-3, "fp32": 2.0e-5}


def check_attention(got, want, dtype, what=""):
    """Asserts |got - want| <= 2^-8 |want| + floor * RMS(want) per element (fp32: the floor alone) and returns the
    measured maxima: absolute, relative to the RMS, and in units of the bound."""
    want = np.asarray(want, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    rms = float(np.sqrt(np.mean(np.square(want))))
    err = np.abs(got - want)
    bound = ATTN_FLOOR_REL[dtype] * rms + (2.0 ** -8 * np.abs(want) if dtype == "bf16" else 0.0)
    m = {"max_abs": float(err.max()), "rms": rms, "max_over_rms": float(err.max() / max(rms, 1e-30)),
         "worst_in_bounds": float((err / bound).max())}
    print("attention", what, {k: float(f"{v:.3g}") for k, v in m.items()})
    assert np.isfinite(got).all()
    assert m["worst_in_bounds"] <= 1.0, (what, m)
    return m


def oracle_num(cfg, big=False):
    return po.Num(np.float32 if big else np.float64, "bf16" if cfg.dtype == "bf16" else "none")


def np_of(t):
    if t.dtype == torch.bfloat16:
        return t.float().cpu().numpy()
    return t.cpu().numpy()


def tree_paths(tokens, parents, n_nodes):
    out = {}
    for r in range(n_nodes):
        p, j = [], r
        while j > 0:
            p.append(int(tokens[j]))
            j = int(parents[j])
        out[tuple(p[::-1])] = r
    return out


def run_gpu_round(P, cfg, kv_np, prefix_len, new_tok, new_feat, depth, K, T):
    from paper_2506_03566_b200.binding import to_device
    dkv = to_device(kv_np)
    tok = torch.from_numpy(np.asarray(new_tok, dtype=np.int32)).cuda()
    feat = to_device(new_feat)
    out = P.poss_draft_round(dkv, prefix_len, tok, feat, depth, K, T)
    n_nodes = int(out["n_nodes"][0])
    tr = P.poss_draft_trace(depth, K, n_nodes)
    torch.cuda.synchronize()
    assert P.poss_last_status() == 0
    host = {k: np_of(v) for k, v in out.items()}
    host["anc_mask"] = host["anc_mask"].view(np.uint64)
    trace = {k: np_of(v) for k, v in tr.items()}
    return host, trace, dkv


def check_structure_self_consistent(g, trace, depth, K, T):
    """What must hold for ANY valid output, from the GPU's own arrays."""
    n = int(g["n_nodes"][0])
    n_cand = K + (depth - 1) * K * K
    assert n == 1 + min(T, n_cand)
    sel = trace["selected"][: n - 1]
    assert np.all(np.diff(sel) > 0)
    assert g["parents"][0] == -1 and g["depth"][0] == 0 and g["scores"][0] == 0
    new_index = {-1: 0}
    for j, c in enumerate(sel):
        new_index[int(c)] = j + 1
    for j, c in enumerate(sel):
        r = j + 1
        assert g["tokens"][r] == trace["cand_tokens"][c]
        assert g["parents"][r] == new_index[int(trace["cand_parents"][c])]      # ancestor-closed
        assert g["scores"][r] == trace["cand_scores"][c]
        lvl = 1 if c < K else 2 + (c - K) // (K * K)
        assert g["depth"][r] == lvl == g["depth"][g["parents"][r]] + 1
        assert g["parents"][r] < r
    want_mask = po.pack_mask(po.ancestor_matrix(g["parents"][:n]))
    words = (T + 1 + 63) // 64
    assert np.array_equal(g["anc_mask"][:n, : want_mask.shape[1]], want_mask)
    assert g["anc_mask"].shape[1] == words


def compare_round(cfg, w, kv_np, prefix_len, new_tok, new_feat, depth, K, T, g, trace, num, require_exact,
                  noise_num=None):
    """Returns a report dict; raises AssertionError on any unexplained difference.  The report carries the measured
    maxima (feature error per step, absolute and relative to the step's RMS; log-prob error) so that a test can
    print them."""
    tol = TOL[cfg.dtype]
    kv_o = po.widen(kv_np, num.dtype).copy()
    free = po.draft_round(cfg, w, kv_o, prefix_len, new_tok, new_feat, depth, K, T, num)
    n = free.n_nodes
    check_structure_self_consistent(g, trace, depth, K, T)
    exact = (len(free.tokens) == n and np.array_equal(free.tokens, g["tokens"][:n]) and np.array_equal(free.parents, g["parents"][:n])
             and np.array_equal(free.depth, g["depth"][:n]) and np.array_equal(free.anc_mask, g["anc_mask"][:n])
             and np.array_equal(free.cand_tok, trace["cand_tokens"]))
    report = {"exact": bool(exact), "inexact_decisions": 0, "min_margin_seen": float("inf")}
    if exact and cfg.dtype == "fp32":
        assert np.abs(free.scores - g["scores"][:n]).max() <= tol * max(depth, 1)
        assert np.abs(free.cand_score - trace["cand_scores"]).max() <= tol * max(depth, 1)
        for i, st in enumerate(free.steps):
            mc = st.fout.shape[0]
            err = np.abs(st.fout - trace["step_features"][i, :mc]).max()
            assert err <= tol, f"step {i} feature error {err}"
            report["max_feature_err"] = max(report.get("max_feature_err", 0.0), float(err))
        report["max_score_err"] = float(np.abs(free.scores - g["scores"][:n]).max())
        kv_final = kv_o
    else:
        assert not require_exact, "check mode must reproduce the oracle's tree exactly"
        # oracle follows the GPU's decisions with its own arithmetic
        top_ids, frontier = [], []
        base = 0
        for i in range(depth):
            mc = 1 if i == 0 else K
            top_ids.append(trace["cand_tokens"][base: base + mc * K].reshape(mc, K))
            base += mc * K
            if i < depth - 1:
                frontier.append(trace["frontier"][i])
        follow = {"top_ids": top_ids, "frontier": frontier, "selected": trace["selected"][: n - 1],
                  "features": [trace["step_features"][i, : (1 if i == 0 else K)] for i in range(depth)],
                  "cand_scores": trace["cand_scores"], "force_head_input": True}
        kv_o = po.widen(kv_np, num.dtype).copy()
        fol = po.draft_round(cfg, w, kv_o, prefix_len, new_tok, new_feat, depth, K, T, num, keep_logits=True,
                             follow=follow)
        kv_final = kv_o
        noise = None
        if noise_num is not None:
            # the same replay in a second precision: how far two correct implementations are apart on this step
            other = po.draft_round(cfg, w, po.widen(kv_np, noise_num.dtype).copy(), prefix_len, new_tok, new_feat, depth,
                                   K, T, noise_num, follow=follow)
            noise = [float(np.abs(np.asarray(a.fout, dtype=np.float64) - b.fout).max())
                     for a, b in zip(other.steps, fol.steps)]
            report["oracle_noise"] = [round(x, 5) for x in noise]
        inexact = 0
        base = 0
        report["feature_err"], report["feature_rms"] = [], []
        for i, st in enumerate(fol.steps):
            mc = st.fout.shape[0]
            err = np.abs(st.fout - trace["step_features"][i, :mc]).max()
            rms = float(np.sqrt(np.mean(np.square(st.fout))))
            report["feature_err"].append(round(float(err), 5))
            report["feature_rms"].append(round(rms, 3))
            ftol = tol
            if noise is not None:
                ftol = min(tol * max(1.0, rms), max(tol, 3.0 * noise[i]))
            assert err <= ftol, f"step {i} feature error {err} > {ftol} (following; RMS {rms})"
            for r in range(mc):
                z = st.logits[r]
                kth = np.sort(z)[-K]
                ids = st.top_ids[r]
                assert len(set(int(t) for t in ids)) == K
                assert np.all(z[ids] >= kth - MARGIN), f"step {i} row {r}: token outside the top-{K} by more than the margin"
                assert np.all(z[ids][:-1] >= z[ids][1:] - MARGIN), f"step {i} row {r}: order off by more than the margin"
                if not np.array_equal(ids, st.own_top_ids[r]):
                    inexact += 1
                    report["min_margin_seen"] = min(report["min_margin_seen"], float(st.row_margin[r]))
            n_step = mc * K
            sc_o = fol.cand_score[base: base + n_step]
            sc_g = trace["cand_scores"][base: base + n_step]
            assert np.abs(sc_o - sc_g).max() <= tol, f"step {i} candidate scores (teacher-forced log-probs)"
            report["max_logp_err"] = max(report.get("max_logp_err", 0.0), float(np.abs(sc_o - sc_g).max()))
            report["max_feature_err"] = max(report.get("max_feature_err", 0.0), float(err))
            if i < depth - 1:
                pick = np.asarray(st.next_frontier) - base
                rest = np.setdiff1d(np.arange(n_step), pick)
                assert len(set(pick.tolist())) == K
                if len(rest):
                    assert sc_o[pick].min() >= sc_o[rest].max() - MARGIN, f"step {i}: frontier not a valid top-{K}"
                assert np.all(sc_o[pick][:-1] >= sc_o[pick][1:] - MARGIN)
                if not np.array_equal(st.next_frontier, st.own_frontier):
                    inexact += 1
                    report["min_margin_seen"] = min(report["min_margin_seen"], float(st.frontier_margin))
            base += n_step
        sel = trace["selected"][: n - 1]
        rest = np.setdiff1d(np.arange(len(fol.cand_score)), sel)
        if len(rest):
            assert fol.cand_score[sel].min() >= fol.cand_score[rest].max() - MARGIN, "rerank not a valid top-T"
        # the oracle's own choice on the teacher-forced scores; those mix the GPU's parent scores with the
        # oracle's log-probs, so when a child's log-prob is ~0 (a near one-hot softmax) a child can tie with
        # or pass its parent and the choice is not ancestor-closed: that is a zero-margin case, not an error
        try:
            own = po.rerank(fol.cand_tok, fol.cand_parent, fol.cand_score, fol.cand_level, int(new_tok[-1]), T)
            own_sel, own_margin = own.selected, float(own.rerank_margin)
        except KeyError:
            own_sel, own_margin = None, 0.0
        if own_sel is None or not np.array_equal(own_sel, sel):
            inexact += 1
            report["min_margin_seen"] = min(report["min_margin_seen"], own_margin)
        assert np.array_equal(fol.tokens, g["tokens"][:n]) and np.array_equal(fol.parents, g["parents"][:n])
        assert np.abs(fol.scores - g["scores"][:n]).max() <= tol
        report["inexact_decisions"] = inexact
        assert report["min_margin_seen"] < MARGIN or inexact == 0, \
            f"GPU decision differs although the oracle margin is {report['min_margin_seen']}"
    report["kv_oracle"] = kv_final
    return report


def compare_kv(cfg, dkv_gpu, kv_oracle, lo, hi, tol):
    got = np_of(dkv_gpu)[:, :, :, lo:hi]
    want = np.asarray(kv_oracle[:, :, :, lo:hi], dtype=np.float64)
    err = np.abs(got - want)
    if cfg.dtype == "bf16":
        # stored values are bf16: allow one unit in the last place where rounding flipped
        ulp = np.maximum(np.abs(want), 1e-30) * 2.0 ** -7
        assert np.all(err <= np.maximum(tol, ulp)), float(err.max())
    else:
        assert err.max() <= tol, float(err.max())
    return float(err.max())


def bonus_is_valid(residual, u, bonus, rel_tol=2e-5):
    """Inverse-CDF draw in fp32 against the fp64 oracle: the threshold u * total must lie in the drawn token's
    cumulative interval up to the rounding of an fp32 sum over the vocabulary (the interval's ends are sums of up to
    128256 terms; in fp32, in the kernel's blocked order, they carry a relative error of the order of 1e-5 of the
    total), and the token must have mass."""
    cdf = np.cumsum(np.asarray(residual, dtype=np.float64))
    total = cdf[-1]
    thr = float(u) * total
    lo = cdf[bonus - 1] if bonus > 0 else 0.0
    return residual[bonus] > 0 and lo - rel_tol * total <= thr <= cdf[bonus] + rel_tol * total
