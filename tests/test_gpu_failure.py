"""Failure detection on the device, without a fault: a bounded wait that runs out.

The tensor-core matrix product waits on shared-memory barriers for its TMA copies and for its own tensor-core
work.  Every such wait gives up after about one second, raises POSS_E_TIMEOUT in the context's status word, and
the CTA leaves in order (copies in flight awaited, tensor memory freed).  The test hook withholds one activation
tile from one launch, so exactly that happens; afterwards the same context must work as before."""
import numpy as np
import pytest
import torch

import poss_synth as ps
from oracle import poss_oracle as po
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    from paper_2506_03566_b200 import Poss, make_config, to_device
    cfg = ps.CONFIGS["t_bf16"].replace(n_target_layers=0)
    P = Poss(make_config(cfg, 512), ps.make_weights(cfg, 1))
    M, N, K = 10, 1408, 512
    x = ps.normal(5, "x", (M, K), 1.0, "bf16")
    W = ps.normal(5, "w", (N, K), 0.02, "bf16")
    xd, Wd = to_device(x), to_device(W)
    want = po.linear(po.widen(x, np.float64), W, pu.oracle_num(cfg))
    good = P.poss_linear(xd, Wd, impl=2).cpu().numpy()
    assert P.poss_last_status() == 0
    assert np.abs(good - want).max() <= 1e-4

    P.poss_debug_lose_load(1)
    P.poss_linear(xd, Wd, impl=2)                  # results undefined; must neither fault nor hang
    torch.cuda.synchronize()
    assert P.poss_last_status() == 6               # POSS_E_TIMEOUT

    P.poss_reset()
    again = P.poss_linear(xd, Wd, impl=2).cpu().numpy()
    assert P.poss_last_status() == 0
    assert np.array_equal(again, good)


def test_the_attention_kernel_reports_a_wait_that_runs_out_and_the_context_stays_usable():
    """The tcgen05 tree attention: its value tiles are never requested, the wait for them runs out, every CTA of
    every cluster still meets its peers at the cluster barrier and leaves in order."""
    import math
    from paper_2506_03566_b200 import Poss, make_config, to_device
    Hq, Hkv, d, rows, P_len = 8, 2, 128, 20, 300
    cfg = ps.CONFIGS["t_bf16"].replace(n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, hidden=Hq * d, vocab=64, ffn=64,
                                       n_target_layers=0)
    P = Poss(make_config(cfg, 64), ps.make_weights(cfg, 1))
    q, kv = ps.make_attention_case(21, rows, Hq, Hkv, d, P_len, P_len + rows + 2, cfg.dtype)
    mask = torch.from_numpy(po.pack_mask(po.ancestor_matrix(ps.random_tree_parents(22, rows))).view(np.int64)).cuda()
    qd, kvd, scale = to_device(q), to_device(kv), 1.0 / math.sqrt(d)
    good = pu.np_of(P.poss_tree_attention(qd, kvd, P_len, mask, scale))
    assert P.poss_last_status() == 0

    P.poss_debug_lose_load(1)
    P.poss_tree_attention(qd, kvd, P_len, mask, scale)      # results undefined; must neither fault nor hang
    torch.cuda.synchronize()
    assert P.poss_last_status() == 6                        # POSS_E_TIMEOUT

    P.poss_reset()
    again = pu.np_of(P.poss_tree_attention(qd, kvd, P_len, mask, scale))
    assert P.poss_last_status() == 0
    assert np.array_equal(again, good)


def test_a_wait_that_runs_out_in_a_counted_product_leaves_no_stale_tile_counters():
    """The LM head with its logits stored runs the matrix product whose split tiles are finished by the last CTA to
    arrive (per-tile arrival counters).  A launch that gives up on a wait may leave counters behind; poss_reset
    clears them, and the same call then reproduces its earlier result bit for bit."""
    from paper_2506_03566_b200 import Poss, make_config, to_device
    cfg = ps.CONFIGS["m_bf16"].replace(S=1, n_target_layers=0)
    P = Poss(make_config(cfg.replace(topk=16, total=16, depth=2), 64), ps.make_weights(cfg, 2))
    f = to_device(ps.normal(4, "f", (10, cfg.hidden), 1.5, "bf16"))
    ids0, logp0, lg0 = P.poss_lm_head_topk(f, 10, want_logits=True)
    assert P.poss_last_status() == 0
    P.poss_debug_lose_load(1)
    P.poss_lm_head_topk(f, 10, want_logits=True)       # results undefined; must neither fault nor hang
    torch.cuda.synchronize()
    assert P.poss_last_status() == 6
    P.poss_reset()
    ids1, logp1, lg1 = P.poss_lm_head_topk(f, 10, want_logits=True)
    assert P.poss_last_status() == 0
    assert torch.equal(ids0, ids1) and torch.equal(logp0, logp1) and torch.equal(lg0, lg1)
