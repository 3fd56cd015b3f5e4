"""The allocation-free block forward (revnet_block_fwd_noalloc) against the regular entry point.

This entry point serves callers that may not allocate device memory (code under a foreign memory
pool, real-time sections, plugins without an allocator): its scratch is a fixed array inside the
library.  The file sorts last on purpose, so that a run that stops at the first failure has already
run every other test."""
import numpy as np
import pytest
import torch

from paper_1707_04585_b200 import binding as B
from paper_1707_04585_b200 import runner as R
from paper_1707_04585_b200 import synthetic as syn

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", [0, 1])
def test_noalloc_block_forward_matches_workspace_version_twice(mode):
    ctx = B.Context(0)
    b = syn.BlockCfg(8, 32, 32, 16, 0, "basic", seed=77)
    for call in range(2):                                   # two calls in a row share the static array
        inp = syn.make_block_inputs(syn.BlockCfg(b.N, b.H, b.W, b.c, b.w, b.kind, seed=77 + call), affine_jitter=True)
        r = R.BlockRunner(ctx, b, mode)
        r.load(inp["params"])
        x1, x2 = R.to_state(inp["x1"], r.frac), R.to_state(inp["x2"], r.frac)
        ref1, ref2 = torch.empty_like(x1), torch.empty_like(x2)
        B.revnet_block_fwd(ctx, r.desc, x1, x2, r.F, r.G, ref1, ref2, r.ws)
        y1, y2 = torch.empty_like(x1), torch.empty_like(x2)
        torch.cuda.synchronize()
        # free device memory as the driver sees it (torch's own counters cannot see what a library allocates)
        free_before = torch.cuda.mem_get_info()[0]
        B.revnet_block_fwd_noalloc(ctx, r.desc, x1, x2, r.F, r.G, y1, y2)
        torch.cuda.synchronize()
        free_after = torch.cuda.mem_get_info()[0]
        if call == 1:
            # the first call on a device may make the runtime place the library's image (with the array) there;
            # from the second call on nothing on the device may change hands
            assert free_after == free_before, (free_before, free_after)
        # same kernels, same order, same inputs: identical bits (well inside the parity tolerances)
        assert torch.equal(y1, ref1) and torch.equal(y2, ref2)
        assert not torch.equal(y1, x1)
    B.revnet_check_device(ctx)
    ctx.close()


def test_noalloc_rejects_shapes_beyond_its_scratch():
    ctx = B.Context(0)
    b = syn.BlockCfg(128, 32, 32, 64, 0, "basic", seed=1)       # needs far more than 16 MiB of scratch
    d = B.block_desc(b, 0, 16)
    t = torch.zeros(16, dtype=torch.int32, device="cuda")
    w = dict(W=t, gamma=t, beta=t)
    with pytest.raises(B.RevnetError, match="static array holds"):
        B.revnet_block_fwd_noalloc(ctx, d, t, t, [w, w], [w, w], t, t)
    ctx.close()
