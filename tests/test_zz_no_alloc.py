"""The allocation-free attention entry point, checked against the regular one through the C ABI.

Collected last on purpose (file name), so a run that stops at the first failure has already run every
other test.  It needs no state from them: it passes alone in a fresh process as well.

Why the entry exists: a caller that is given device pointers but is not allowed to allocate -- pools
sized at start-up, a stream that must not hit cudaMalloc's implicit synchronisation, a plugin without
the host's allocator -- cannot build the workspace a context needs.  poss_tree_attention_noalloc keeps
its split-KV partials in a fixed array inside the library instead.
"""
import math

import numpy as np
import pytest
import torch

import poss_synth as ps
from oracle import poss_oracle as po
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def _case(seed, rows, prefix, hq, hkv, d, dtype):
    from paper_2506_03566_b200 import to_device
    cap = prefix + rows + 2
    q, kv = ps.make_attention_case(seed, rows, hq, hkv, d, prefix, cap, dtype)
    parents = ps.random_tree_parents(seed, rows)
    anc = np.zeros((rows, (rows + 63) // 64), dtype=np.uint64)
    for r in range(rows):
        j = r
        while j >= 0:
            anc[r, j // 64] |= np.uint64(1) << np.uint64(j % 64)
            j = int(parents[j])
    want = po.tree_attention(q, kv, prefix, parents, 1.0 / math.sqrt(d), po.Num(np.float64, "bf16" if dtype == "bf16" else "none"))
    return to_device(q), to_device(kv), torch.from_numpy(anc.view(np.int64)).cuda(), want


@pytest.mark.parametrize("dtype,d,tol", [("bf16", 64, 2e-2), ("bf16", 128, 2e-2), ("fp32", 64, 1e-5)])
def test_noalloc_attention_equals_the_context_entry_on_two_calls_in_a_row(dtype, d, tol):
    """Against the regular entry point (within the tolerance of the other attention tests; at head dimension 128
    the regular entry runs another kernel, which groups its sums differently) and, element by element, against
    the CPU oracle."""
    from paper_2506_03566_b200 import Poss, make_config
    from paper_2506_03566_b200.binding import poss_tree_attention_noalloc
    hq, hkv = 8, 2
    cfg = ps.CONFIGS["t_bf16" if dtype == "bf16" else "t_fp32"].replace(
        n_q_heads=hq, n_kv_heads=hkv, head_dim=d, hidden=hq * d, vocab=64, ffn=64, n_target_layers=0)
    P = Poss(make_config(cfg, 64), ps.make_weights(cfg, 1))
    scale = 1.0 / math.sqrt(d)
    # two different problems back to back: the second must not see the first one's leftovers
    for call, (seed, rows, prefix) in enumerate([(51, 61, 1500), (52, 23, 200)]):
        q, kv, mask, oracle = _case(seed, rows, prefix, hq, hkv, d, dtype)
        want = P.poss_tree_attention(q, kv, prefix, mask, scale)
        out = torch.empty_like(q)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        poss_tree_attention_noalloc(q, kv, prefix, mask, scale, out)
        torch.cuda.synchronize()
        if call > 0:        # the first call may load the kernels' code; after that the device's free memory stays put
            assert torch.cuda.mem_get_info()[0] == free_before
        assert torch.isfinite(out.float()).all()
        assert (out.float() - want.float()).abs().max().item() <= tol
        pu.check_attention(pu.np_of(out), oracle, dtype, f"no-alloc d{d} {rows}x{prefix}")
        pu.check_attention(pu.np_of(want), oracle, dtype, f"context entry d{d} {rows}x{prefix}")


def test_noalloc_attention_rejects_what_does_not_fit():
    from paper_2506_03566_b200.binding import PossError, poss_tree_attention_noalloc
    # 128 rows x 128 heads x (128+2) floats = 2.13M floats > the 2,097,152-float array
    rows, hq, d = 128, 128, 128
    q = torch.zeros((rows, hq, d), dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros((2, 16, rows + 1, d), dtype=torch.bfloat16, device="cuda")
    mask = torch.zeros((rows, 2), dtype=torch.int64, device="cuda")
    with pytest.raises(PossError) as e:
        poss_tree_attention_noalloc(q, kv, 0, mask, 1.0, torch.empty_like(q))
    assert e.value.code == 3
    # tensors that do not start on a 16-byte boundary are refused on the host, not faulted on in a kernel
    q8 = torch.zeros((9, 8, 64), dtype=torch.bfloat16, device="cuda")
    kv8 = torch.zeros((2, 2, 16, 64), dtype=torch.bfloat16, device="cuda")
    m8 = torch.ones((8, 1), dtype=torch.int64, device="cuda")
    off = q8.view(-1)[1:1 + 8 * 8 * 64].view(8, 8, 64)          # one element (2 bytes) past the boundary
    lib = __import__("paper_2506_03566_b200.binding", fromlist=["load_library"]).load_library()
    rc = lib.poss_tree_attention_noalloc(off.data_ptr(), kv8.data_ptr(), 16, 0, 8, 8, 2, 64, 1, m8.data_ptr(), 1.0,
                                         q8.data_ptr(), torch.cuda.current_stream().cuda_stream)
    assert rc == 1
