"""The chunked refresh kernel hands data between four warp roles through mbarriers, tensor memory and shared
memory.  A missing or misplaced hand-off would show as run-to-run differences long before it shows as a tolerance
failure, so the same launch is repeated and its results compared bit for bit (one issuing thread, fixed
accumulation order: the kernel is deterministic by construction)."""
import numpy as np
import pytest
import torch

import paper_2608_30386_b200 as dasc
from helpers import make_refresh_case, run_refresh_gpu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("kind,H_k,with_o", [(dasc.KDA, 8, True), (dasc.KDA, 8, False), (dasc.GDN, 4, True)])
def test_repeated_launches_give_identical_bits(kind, H_k, with_o):
    # 12 requests x 2 layers x 8 heads = 192 CTAs of mixed length (1 to 9 chunks, ragged tails): more CTAs than fit
    # on the GPU at once would only add waves; what matters is many chunk hand-offs with two CTAs sharing an SM
    lens = [257, 32, 1, 100, 288, 64, 31, 200, 33, 96, 150, 7]
    case = make_refresh_case(41, kind, 2, 8, H_k, 128, 128, lens, scope=dasc.SCOPE_LAYER, keep_ratio=0.38)
    first_s, first_o = run_refresh_gpu(case, algo=dasc.ALGO_CHUNKED, want_o=with_o, o_dtype=torch.bfloat16)
    for _ in range(7):
        s, o = run_refresh_gpu(case, algo=dasc.ALGO_CHUNKED, want_o=with_o, o_dtype=torch.bfloat16)
        np.testing.assert_array_equal(s.view(np.uint32), first_s.view(np.uint32))
        if with_o:
            np.testing.assert_array_equal(o, first_o)
