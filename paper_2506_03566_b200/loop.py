"""Host driver of the full draft-then-verify loop; every step is a call into the C library."""
from __future__ import annotations

import torch


def speculative_generate(P, prompt, n_generate, depth, topk, total, log=None, temperature=0.0, generator=None):
    """Speculative decoding: prefill, then rounds of
    poss_draft_round -> poss_target_forward (tree-masked) -> poss_verify_accept -> poss_kv_compact.
    temperature 0: greedy verification.  temperature > 0: the target pass also returns its logits and
    poss_verify_sample walks the tree by rejection sampling with uniforms drawn from `generator` (a CUDA
    torch.Generator; the first token after the prompt is drawn the same way, from a one-row tree).

    P: binding.Poss with target layers; prompt: int32 CUDA tensor.  Returns a list of n_generate ids.
    The accepted length is read back once per round (the emitted tokens leave the device anyway)."""
    n = int(prompt.numel())
    n_cand = topk + (depth - 1) * topk * topk
    assert n_cand >= total, "the loop hands fixed-size trees to the target"
    rows = total + 1
    sampling = temperature > 0.0
    tkv = P.new_target_kv()
    dkv = P.new_draft_kv()
    if not sampling:
        feats, arg = P.poss_target_prefill(tkv, 0, prompt)
        new_tok = arg[n - 1:n].clone()
        new_feat = feats[n - 1:n].clone()
    else:
        feats = torch.empty((n, P.config.hidden), dtype=P.dtype, device="cuda")
        if n > 1:
            feats[: n - 1], _ = P.poss_target_prefill(tkv, 0, prompt[: n - 1].contiguous())
        zero = torch.zeros(1, dtype=torch.int32, device="cuda")
        one = torch.ones(1, dtype=torch.int64, device="cuda")
        f_last, _, lg = P.poss_target_forward(tkv, n - 1, prompt[n - 1:].contiguous(), zero, one, 1, want_logits=True)
        feats[n - 1:] = f_last
        root_only = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        u = torch.rand(2, device="cuda", generator=generator)
        first = P.poss_verify_sample(lg, f_last, prompt[n - 1:].contiguous(), root_only, 1, temperature, u)
        new_tok = first["new_tokens"][:1].contiguous()
        new_feat = first["new_features"][:1].contiguous()
    if n > 1:
        # drafter pair j = [token j+1 ; feature j]
        P.poss_draft_prefill(dkv, 0, prompt[1:].contiguous(), feats[:-1].contiguous())
    out = [int(new_tok[0])]
    p_target, p_draft = n, n - 1
    while len(out) < n_generate:
        tree = P.poss_draft_round(dkv, p_draft, new_tok, new_feat, depth, topk, total)
        tf, targ, lg = P.poss_target_forward(tkv, p_target, tree["tokens"], tree["depth"], tree["anc_mask"], rows,
                                             want_logits=sampling)
        if sampling:
            u = torch.rand(rows, device="cuda", generator=generator)
            va = P.poss_verify_sample(lg, tf, tree["tokens"], tree["parents"], rows, temperature, u)
        else:
            va = P.poss_verify_accept(None, targ, tf, tree["tokens"], tree["parents"], rows)
        P.poss_kv_compact(tkv, p_target, va["path"], va["n_accepted"])
        a = int(va["n_accepted"][0])
        new_tok = va["new_tokens"][: a + 1].contiguous()
        new_feat = va["new_features"][: a + 1].contiguous()
        out.extend(int(t) for t in new_tok.tolist())
        if log is not None:
            log.append((a, va["path"][: a + 1].tolist()))
        p_draft = p_target
        p_target += a + 1
    return out[:n_generate]


def plain_generate(P, prompt, n_generate):
    """Vanilla greedy decoding of the target with the same kernels, one row per step."""
    n = int(prompt.numel())
    tkv = P.new_target_kv()
    feats, arg = P.poss_target_prefill(tkv, 0, prompt)
    cur = arg[n - 1:n].clone()
    out = [int(cur[0])]
    p = n
    while len(out) < n_generate:
        _, cur = P.poss_target_prefill(tkv, p, cur)
        out.append(int(cur[0]))
        p += 1
    return out
