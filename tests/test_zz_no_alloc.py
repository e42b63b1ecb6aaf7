"""The allocation-free layout entry point, for embedders that may not call cudaMalloc (code inside another
framework's memory pool, runtimes that own all device memory): its scratch is a fixed array inside the
library.  Checked against the context-based entry point, bit for bit, on two calls in a row -- the second
with different inputs, so that whatever the first call left in the shared scratch would show."""
import pytest
import torch

from paper_2609_00993_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _reference_layout(idx, E):
    T, k = idx.shape
    ctx = B.MoeContext(B.make_config(256, E, k, 128, 0, max(T, 1)))
    bufs = B.alloc_step_buffers(T, k, E, DEV)
    torch.cuda.synchronize()
    ctx.moe_dispatch_layout(idx, None, bufs["counts"], bufs["offsets"], bufs["perm"], bufs["inv_perm"], T=T)
    torch.cuda.synchronize()
    ctx.close()
    return bufs


def _random_idx(T, E, k, seed):
    g = torch.Generator(device=DEV).manual_seed(seed)
    pop = torch.rand(E, generator=g, device=DEV) ** 3 + 1e-4
    return torch.multinomial(pop.expand(T, E), k, replacement=False, generator=g).to(torch.int32)


@pytest.mark.parametrize("T,E,k", [(5000, 256, 8),   # multi-CTA path: uses the scratch array
                                   (100, 64, 4)])    # single-CTA path
def test_static_layout_matches_context_layout_twice(T, E, k):
    for call, seed in enumerate((11, 12)):
        idx = _random_idx(T, E, k, seed)
        want = _reference_layout(idx, E)
        got = B.alloc_step_buffers(T, k, E, DEV)
        for t in got.values():
            t.fill_(-7) if t.dtype == torch.int32 else None
        torch.cuda.synchronize()
        st = B.moe_dispatch_layout_static(idx, E, got["counts"], got["offsets"], got["perm"], got["inv_perm"])
        torch.cuda.synchronize()
        assert st == B.MOE_OK, f"call {call}: status {st}"
        for name in ("counts", "offsets", "perm", "inv_perm"):
            assert torch.equal(got[name], want[name]), f"call {call}: {name} differs"


def test_static_layout_rejects_sizes_beyond_its_scratch():
    E, k = 1024, 8
    T = 66 * 1024 // k  # 66 chunks * 1024 experts > 65536 cells
    idx = torch.zeros(T, k, dtype=torch.int32, device=DEV)
    b = B.alloc_step_buffers(T, k, E, DEV)
    st = B.moe_dispatch_layout_static(idx, E, b["counts"], b["offsets"], b["perm"], b["inv_perm"])
    assert st == B.MOE_ERR_CAPACITY
    assert B.moe_dispatch_layout_static(idx[:16], 2000, b["counts"], b["offsets"], b["perm"], b["inv_perm"]) \
        == B.MOE_ERR_INVALID_ARG
