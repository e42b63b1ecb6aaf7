"""Property tests of the oracle's integer stages (hypothesis): the invariants that make the routing indices and the
layout unique hold on arbitrary, tie-heavy inputs, and the layout agrees with a brute-force stable sort."""
import numpy as np
from hypothesis import given, settings
from hypothesis import strategies as st

import oracle


@settings(max_examples=60, deadline=None)
@given(st.integers(1, 24), st.integers(1, 40), st.data())
def test_route_is_the_unique_lexicographic_top_k(T, E, data):
    k = data.draw(st.integers(1, E))
    # few distinct values (multiples of 0.5, both zeros) so that ties are the rule
    vals = data.draw(st.lists(st.sampled_from([-1.0, -0.5, -0.0, 0.0, 0.5, 1.0]), min_size=T * E, max_size=T * E))
    logits = np.array(vals, np.float32).reshape(T, E)
    idx, w = oracle.route(logits, None, k)
    for t in range(T):
        order = sorted(range(E), key=lambda e: (-float(logits[t, e]), e))
        assert idx[t].tolist() == order[:k]
        assert abs(float(w[t].sum()) - 1.0) < 1e-5
        sel = logits[t, idx[t]].astype(np.float64)
        ref = np.exp(sel - sel.max())
        assert np.allclose(w[t], ref / ref.sum(), rtol=1e-6)


@settings(max_examples=80, deadline=None)
@given(st.integers(0, 300), st.integers(1, 33), st.data())
def test_layout_is_the_stable_counting_sort(N, E, data):
    idx = np.array(data.draw(st.lists(st.integers(0, E - 1), min_size=N, max_size=N)), np.int32)
    counts, offsets, perm, inv = oracle.layout(idx, E)
    assert counts.tolist() == [int((idx == e).sum()) for e in range(E)]
    assert offsets.tolist() == [int((idx < e).sum()) for e in range(E + 1)]
    brute = sorted(range(N), key=lambda f: (int(idx[f]), f))
    assert perm.tolist() == brute
    assert all(inv[perm[p]] == p for p in range(N))
