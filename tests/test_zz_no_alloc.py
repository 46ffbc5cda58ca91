"""The backward for callers that cannot allocate device memory (`seg_attn_bwd_static`): same results
as `seg_attn_bwd`, with the row dots kept in the library's fixed device array instead of a
caller-provided workspace.  Collected last on purpose, so that a run stopping at the first failure has
already run every other test; passes alone in a fresh process and after the rest of the suite."""
import pytest
import torch

import oracle
import paper_2605_11744_b200 as sa
from util import TOL_GRAD, assert_grads_close, f64, rand_inputs, rel_l2

pytestmark = pytest.mark.gpu


def _both_ways(B, L, Hq, Hkv, d, S, T, mask, seed):
    Q, K, V, dO = rand_inputs(B, L, Hq, Hkv, d, seed=seed)
    O, LSE = sa.seg_attn_fwd(Q, K, V, S, T, mask)
    ref = sa.seg_attn_bwd(Q, K, V, O, LSE, dO, S, T, mask)
    # caller-owned gradient buffers, pre-filled so that stale contents would show
    outs = tuple(torch.full_like(t, float("nan")) for t in (Q, K, V))
    got = sa.seg_attn_bwd_static(Q, K, V, O, LSE, dO, S, T, mask, out=outs)
    sa.poll_status()
    # and against the fp64 oracle directly, not only through the other entry point
    assert_grads_close(got, oracle.bwd(f64(Q), f64(K), f64(V), f64(dO), S, T, mask), "static scratch vs oracle")
    return ref, got


def test_static_scratch_backward_matches_workspace_backward_twice_in_a_row():
    # the second call is smaller than the first, so most of the shared array still holds the first call's row dots
    for B, L, Hq, Hkv, d, S, T, mask, seed in ((2, 1024, 4, 2, 128, 256, 128, [0, 1], 21),
                                               (1, 333, 2, 2, 64, 100, 100, [1, 0], 22)):
        ref, got = _both_ways(B, L, Hq, Hkv, d, S, T, mask, seed)
        for name, a, b in zip(("dQ", "dK", "dV"), got, ref):
            assert torch.isfinite(a.float()).all(), name
            assert rel_l2(f64(a), f64(b)) <= TOL_GRAD, name
            assert torch.equal(a, b), name + ": same kernels, same order of arithmetic"


def test_problems_larger_than_the_fixed_scratch_are_rejected_before_launch():
    rows = sa.binding.STATIC_MAX_ROWS
    L = rows // 2 + 128                       # B * Hq * Lq = 2 * L > the limit
    mk = lambda H: torch.zeros(1, L, H, 64, dtype=torch.bfloat16, device="cuda")
    Q, K, V = mk(2), mk(1), mk(1)
    LSE = torch.zeros(1, 2, L, dtype=torch.float32, device="cuda")
    sentinel = tuple(torch.full_like(t, 7.0) for t in (Q, K, V))
    with pytest.raises(sa.SegAttnError) as e:
        sa.seg_attn_bwd_static(Q, K, V, Q, LSE, Q, 128, 0, [0], out=sentinel)
    assert e.value.status == 6 and "SEG_ATTN_STATIC_MAX_ROWS" in str(e.value)
    torch.cuda.synchronize()
    assert all(bool((t == 7.0).all()) for t in sentinel)   # nothing was launched
