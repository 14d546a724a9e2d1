"""The allocation-free page selection (gkv_quest_select_static) must return exactly what
gkv_quest_select returns.  It exists for callers that cannot let the library's work depend on any
device allocation (a fixed arena inside a fully committed memory pool, a no-allocation real-time
loop), so its score scratch is a fixed array inside the library.  Two calls in a row: the array
keeps the first call's scores, and the second call must not be disturbed by them."""
import dataclasses

import pytest
import torch

from paper_2608_23599_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_static_scratch_selection_matches_arena_selection_twice():
    from paper_2608_23599_b200 import binding as B
    B.build()
    w = W.config(3, "small")
    cache = B.Cache(B.config_from_workload(w))
    dev = cache.device
    data = W.make_layer(w, 0, "cpu")
    cache.gkv_append_demote(0, data["k"].to(dev), data["v"].to(dev), token_mass=data["mass"].to(dev))
    k = w.quest_budget_tokens // w.page_tokens
    gen = torch.Generator(device="cpu")
    gen.manual_seed(77)
    # two calls in a row with different queries: the second one sees the first one's leftovers
    # in the shared array and must not be influenced by them
    for call in range(2):
        q = data["q"] if call == 0 else torch.randn(data["q"].shape, generator=gen).to(torch.bfloat16)
        q = q.to(dev)
        want = torch.full((w.batch, w.n_kv_heads, k), -1, dtype=torch.int32, device=dev)
        got = torch.full((w.batch, w.n_kv_heads, k), -2, dtype=torch.int32, device=dev)
        n_want = cache.gkv_quest_select(0, q, w.quest_budget_tokens, want)
        n_got = cache.gkv_quest_select_static(0, q, w.quest_budget_tokens, got)
        torch.cuda.synchronize()
        assert n_got == n_want == k
        assert torch.equal(got, want), f"call {call}: selected pages differ"
    # a smaller budget after a larger one (fewer pages kept, same scores scratch)
    small_want = torch.zeros((w.batch, w.n_kv_heads, 4), dtype=torch.int32, device=dev)
    small_got = torch.zeros_like(small_want)
    assert cache.gkv_quest_select(0, q, 4 * w.page_tokens, small_want) == 4
    assert cache.gkv_quest_select_static(0, q, 4 * w.page_tokens, small_got) == 4
    torch.cuda.synchronize()
    assert torch.equal(small_got, small_want)
    cache.close()


def test_static_scratch_rejects_sizes_beyond_its_maximum():
    """More page scores than the fixed array holds (1,048,576) -> GKV_ERR_UNSUPPORTED, while the
    arena-backed call still works on the same cache."""
    from paper_2608_23599_b200 import binding as B
    B.build()
    if torch.cuda.get_device_properties(0).total_memory < 60e9:
        pytest.skip("needs ~20 GB of device memory")
    # 512 streams x 2056 closed pages (padded) = 1,052,672 scores; every block is a centroid so the
    # cache itself stays small
    T = 2052 * 16
    w = W.Workload("too_many_pages", 7, 1, 64, 32, 8, 128, 128, T, T + 64, page_tokens=16,
                   stair_tokens=(0, 0, 0, 0))
    cache = B.Cache(B.config_from_workload(w))
    dev = cache.device
    g = torch.Generator(device=dev)
    g.manual_seed(5)
    k = torch.randn((w.batch, T, w.n_kv_heads, 128), generator=g, device=dev, dtype=torch.bfloat16)
    v = torch.randn((w.batch, T, w.n_kv_heads, 128), generator=g, device=dev, dtype=torch.bfloat16)
    q = torch.randn((w.batch, w.n_q_heads, 128), generator=g, device=dev, dtype=torch.bfloat16)
    cache.gkv_append_demote(0, k, v)
    del k, v
    pages = torch.zeros((w.batch, w.n_kv_heads, 8), dtype=torch.int32, device=dev)
    with pytest.raises(B.GkvError) as e:
        cache.gkv_quest_select_static(0, q, 8 * 16, pages)
    assert e.value.status == -5
    assert cache.gkv_quest_select(0, q, 8 * 16, pages) == 8
    torch.cuda.synchronize()
    assert int(pages.min()) >= 0 and int(pages.max()) < 2052
    cache.close()
