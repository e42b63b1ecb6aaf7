"""The allocation-free layout entry point, for embedders that may not call cudaMalloc (code inside another
framework's memory pool, runtimes that own all device memory): its scratch is a fixed array inside the
library.  Checked against the context-based entry point, bit for bit, on two calls in a row -- the second
with different inputs, so that whatever the first call left in the shared scratch would show -- and against the
CPU oracle's layout, since the two entry points run the same kernels."""
import numpy as np
import pytest
import torch

import oracle
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
        ref = dict(zip(("counts", "offsets", "perm", "inv_perm"), oracle.layout(idx.cpu().numpy().reshape(-1), E)))
        for name in ("counts", "offsets", "perm", "inv_perm"):
            assert np.array_equal(got[name].cpu().numpy(), ref[name]), f"call {call}: {name} differs from the oracle"


def test_static_layout_at_its_capacity_boundary_empty_batch_and_bad_index():
    # exactly 65536 scratch cells: 256 chunks of 256 slots x 256 experts
    E, k = 256, 8
    T = 256 * 256 // k
    idx = _random_idx(T, E, k, 13)
    got = B.alloc_step_buffers(T, k, E, DEV)
    assert B.moe_dispatch_layout_static(idx, E, got["counts"], got["offsets"], got["perm"], got["inv_perm"]) == B.MOE_OK
    torch.cuda.synchronize()
    ref = dict(zip(("counts", "offsets", "perm", "inv_perm"), oracle.layout(idx.cpu().numpy().reshape(-1), E)))
    for name in ("counts", "offsets", "perm", "inv_perm"):
        assert np.array_equal(got[name].cpu().numpy(), ref[name]), name
    # one slot more than that is refused
    more = B.alloc_step_buffers(T + 1, k, E, DEV)
    idx1 = torch.cat([idx, idx[:1]])
    assert B.moe_dispatch_layout_static(idx1, E, more["counts"], more["offsets"], more["perm"], more["inv_perm"]) \
        == B.MOE_ERR_CAPACITY
    # an empty batch zero-fills counts and offsets
    got["counts"].fill_(-1); got["offsets"].fill_(-1)
    assert B.moe_dispatch_layout_static(idx[:0], E, got["counts"], got["offsets"], got["perm"], got["inv_perm"], T=0,
                                        top_k=k) == B.MOE_OK
    torch.cuda.synchronize()
    assert torch.all(got["counts"] == 0) and torch.all(got["offsets"] == 0)
    # an expert index outside [0, E) is dropped: inv_perm = -1 for that slot, the others laid out as if it were absent
    for T2 in (100, 5000):  # single-CTA and multi-CTA path
        bad = _random_idx(T2, E, k, 14)
        bad[7, 3] = E + 5
        bad[T2 - 1, 0] = -2
        g2 = B.alloc_step_buffers(T2, k, E, DEV)
        assert B.moe_dispatch_layout_static(bad, E, g2["counts"], g2["offsets"], g2["perm"], g2["inv_perm"]) == B.MOE_OK
        torch.cuda.synchronize()
        flat = bad.cpu().numpy().reshape(-1)
        ok = (flat >= 0) & (flat < E)
        c, o, p, inv = oracle.layout(flat[ok], E)           # the valid slots alone
        kept = np.nonzero(ok)[0]
        assert np.array_equal(g2["counts"].cpu().numpy(), c) and np.array_equal(g2["offsets"].cpu().numpy(), o)
        n_ok = int(ok.sum())
        assert np.array_equal(g2["perm"].cpu().numpy()[:n_ok], kept[p])
        want_inv = np.full(flat.size, -1, np.int32)
        want_inv[kept] = inv
        assert np.array_equal(g2["inv_perm"].cpu().numpy(), want_inv)


def test_static_layout_rejects_sizes_beyond_its_scratch():
    E, k = 1024, 8
    T = 66 * 1024 // k  # 66 chunks * 1024 experts > 65536 cells
    idx = torch.zeros(T, k, dtype=torch.int32, device=DEV)
    b = B.alloc_step_buffers(T, k, E, DEV)
    st = B.moe_dispatch_layout_static(idx, E, b["counts"], b["offsets"], b["perm"], b["inv_perm"])
    assert st == B.MOE_ERR_CAPACITY
    assert B.moe_dispatch_layout_static(idx[:16], 2000, b["counts"], b["offsets"], b["perm"], b["inv_perm"]) \
        == B.MOE_ERR_INVALID_ARG
