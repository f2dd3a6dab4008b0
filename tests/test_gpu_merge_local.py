"""GPU-vs-oracle parity of the token merge with the matching kept inside nearby partition blocks
(the local reading of Sec. 3.3).  Same gates as the global merge: integer outputs identical to the
oracle's outside the near-tie band, cosines within 2e-6, merged features within one bf16 ulp."""
import numpy as np
import pytest
import torch

import oracle
from parity_utils import bf16_ulp_distance, bits, check_merge_plan

DEV = "cuda:0"


@pytest.fixture(scope="module")
def usv():
    import paper_2512_05754_b200 as m
    return m


def _rand_bf16(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(shape, generator=g) * scale).to(torch.bfloat16)


CASES = [
    # grid, partition, window, C, Hm, dm, B, r values
    ((4, 6, 8), (1, 1, 2), (1, 1, 1), 64, 2, 64, 2, [0, 40, 96]),
    ((5, 9, 10), (2, 2, 2), (1, 2, 0), 72, 3, 128, 1, [100, 375]),     # ragged blocks, a flat window
    ((6, 20, 32), (1, 1, 2), (0, 0, 0), 128, 2, 128, 1, [1920]),        # own block only, every source merges
    ((6, 20, 32), (1, 2, 2), (1, 1, 1), 256, 4, 128, 2, [1000, 2880]),  # several launch blocks per batch element
    ((21, 30, 52), (1, 1, 2), (1, 1, 1), 256, 12, 128, 1, [16380]),     # the Wan 480p grid and head count, every source merges
]


@pytest.mark.gpu
@pytest.mark.parametrize("case", CASES, ids=["g%dx%dx%d_w%d%d%d" % (c[0] + c[2]) for c in CASES])
def test_local_merge_matches_the_oracle(usv, case):
    grid, part, win, C, Hm, dm, B, rs = case
    N = grid[0] * grid[1] * grid[2]
    x = _rand_bf16((B, N, C), 41)
    metric = _rand_bf16((B, N, Hm, dm), 42)
    is_dst = oracle.destination_mask(grid, part)
    nA = int((~is_dst).sum())
    for r in rs:
        assert r <= nA
        xm, plan = usv.token_merge(x.to(DEV), metric.to(DEV), grid, part, r, debug=True, window=win)
        torch.cuda.synchronize()
        pg = dict(dst_of=plan.dst_of.cpu().numpy(), pos=plan.pos.cpu().numpy(),
                  u=plan.u.cpu().numpy(), jstar=plan.jstar.cpu().numpy())
        stats = check_merge_plan(pg, metric, grid, part, r, window=win)
        print("window %s r=%d: %s" % (win, r, stats))
        ref = oracle.round_to_bf16(oracle.merge_apply(x, pg["dst_of"], pg["pos"], N - r))
        assert bf16_ulp_distance(bits(xm), ref).max() <= 1
        y = usv.token_unmerge(xm, plan.pos)
        assert np.array_equal(bits(y), oracle.unmerge(bits(xm), pg["pos"]))


@pytest.mark.gpu
def test_a_window_over_the_whole_grid_gives_the_global_merge(usv):
    grid, part = (4, 6, 8), (1, 2, 2)
    N = 4 * 6 * 8
    x = _rand_bf16((1, N, 64), 51).to(DEV)
    metric = _rand_bf16((1, N, 2, 128), 52).to(DEV)
    xm_g, plan_g = usv.token_merge(x, metric, grid, part, 60, debug=True)
    xm_l, plan_l = usv.token_merge(x, metric, grid, part, 60, debug=True, window=(4, 3, 4))
    torch.cuda.synchronize()
    assert torch.equal(plan_g.dst_of, plan_l.dst_of) and torch.equal(plan_g.pos, plan_l.pos)
    assert torch.equal(xm_g, xm_l)


@pytest.mark.gpu
def test_negative_window_is_rejected(usv):
    x = torch.zeros(1, 24, 64, dtype=torch.bfloat16, device=DEV)
    m = torch.zeros(1, 24, 1, 64, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(usv.USVError) as e:
        usv.token_merge(x, m, (2, 3, 4), (1, 1, 2), 3, window=(0, -1, 0))
    assert e.value.status == 1
