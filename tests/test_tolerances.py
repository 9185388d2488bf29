"""Where the bf16 tolerances of the parity tests come from: a measurement, on the CPU, of how far two CORRECT
implementations of the same round are apart.  Both are the oracle under the bf16 precision contract (activation
operands and cache entries rounded to bf16), one with fp32 and one with fp64 arithmetic between the rounding points.
They differ wherever an fp32-level difference flips a bf16 rounding, and every flip is a whole bf16 unit of that
element.  The CUDA path (fp32 accumulation in yet another order) sits at the same kind of distance from either."""
import numpy as np

import poss_synth as ps
from oracle import poss_oracle as po
from tests import parity_util as pu


def _two_oracles(name, seed, n_new, force_head_input):
    cfg = ps.CONFIGS[name].replace(n_target_layers=0)
    w = ps.make_weights(cfg, seed)
    cap = cfg.prefix + n_new + cfg.tree_slots
    kv = ps.make_draft_kv(cfg, seed, cap)
    tok, feat = ps.make_round_inputs(cfg, seed, n_new)
    n64, n32 = po.Num(np.float64, "bf16"), po.Num(np.float32, "bf16")
    a = po.draft_round(cfg, w, po.widen(kv, np.float64).copy(), cfg.prefix, tok, feat, cfg.depth, cfg.topk, cfg.total,
                       n64, keep_logits=True)
    # the fp32 oracle replays the fp64 oracle's decisions from its per-step features and parent scores: the per-step,
    # teacher-forced comparison the GPU tests make
    follow = {"top_ids": [st.top_ids for st in a.steps], "frontier": [st.next_frontier for st in a.steps[:-1]],
              "selected": a.selected, "features": [st.fout for st in a.steps], "cand_scores": a.cand_score,
              "force_head_input": force_head_input}
    b = po.draft_round(cfg, w, po.widen(kv, np.float32).copy(), cfg.prefix, tok, feat, cfg.depth, cfg.topk, cfg.total,
                       n32, keep_logits=True, follow=follow)
    return a, b


def test_bf16_tolerances_sit_above_the_distance_between_two_correct_implementations():
    a, b = _two_oracles("m_bf16", 12, 1, True)
    feat_noise, logit_noise, rms = [], [], []
    for sa, sb in zip(a.steps, b.steps):
        feat_noise.append(float(np.abs(sa.fout - sb.fout).max()))
        logit_noise.append(float(np.abs(sa.logits - sb.logits).max()))
        rms.append(float(np.sqrt(np.mean(sa.fout ** 2))))
    print("m_bf16 per step: feature RMS", np.round(rms, 3), "fp32/fp64 feature distance", np.round(feat_noise, 5),
          "logit distance on identical head inputs", np.round(logit_noise, 8))
    # features: flips of whole bf16 units are there (far above fp32 rounding) and the 2e-2 bound leaves them a factor
    # of at least 3, at most 30: wide enough for two correct implementations, narrow enough to bite
    assert max(feat_noise) > 1e-4
    assert 3.0 * max(feat_noise) <= pu.TOL["bf16"] <= 30.0 * max(feat_noise)
    # the LM head on identical inputs: nothing is rounded between the feature and the log-probs, so the two agree to
    # fp32 rounding
    assert max(logit_noise) < 1e-5


def test_the_head_is_compared_on_identical_inputs_because_its_input_rounding_flips():
    """Without forcing the head's input, each side rounds ITS OWN feature to bf16 before the LM head: features that
    agree to ~1e-3 round differently in some elements and the logits move by far more than on identical inputs.
    That, not an error of either side, is why the parity tests compare the feature and the head separately."""
    a, b = _two_oracles("m_bf16", 12, 1, False)
    own = max(float(np.abs(sa.logits - sb.logits).max()) for sa, sb in zip(a.steps, b.steps))
    a2, b2 = _two_oracles("m_bf16", 12, 1, True)
    forced = max(float(np.abs(sa.logits - sb.logits).max()) for sa, sb in zip(a2.steps, b2.steps))
    print("logit distance, each head on its own feature:", own, "on identical inputs:", forced)
    assert own > 100.0 * forced
