"""The routing-plan entry point that allocates nothing (moe_plan_routing_static).

Some users of the library cannot call cudaMalloc where they need a routing plan (the device already belongs
to another memory pool, or their hook is not allowed to allocate), so this entry point keeps its scratch in a
fixed array inside the library instead of in a context.  The test calls it through the C ABI twice in a row,
with different inputs, and checks each result against the context-based moe_plan_routing (same kernels, so
the integer outputs must be identical and the weights equal to the last bit).  It lives in a file pytest
collects last; it must pass alone in a fresh process and after all other tests."""
import numpy as np
import pytest
import torch

from paper_2607_23264_b200 import binding

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _buffers(T, E, k):
    i32 = dict(dtype=torch.int32, device=DEV)
    R = T * k
    return dict(topk_ids=torch.full((R,), -1, **i32), topk_w=torch.full((R,), float("nan"), device=DEV),
                counts=torch.full((E,), -1, **i32), offsets=torch.full((E + 1,), -1, **i32),
                perm=torch.full((R,), -1, **i32), inv_perm=torch.full((R,), -1, **i32))


def _plan_with_context(T, E, k, logits):
    ctx = binding.Context(T, 64, 64, E, k)
    b = _buffers(T, E, k)
    ctx.moe_plan_routing(logits, **b)
    torch.cuda.synchronize()
    return b


@pytest.mark.parametrize("T,E,k", [(1000, 64, 4), (4096, 256, 8)])
def test_static_scratch_plan_matches_context_plan_twice(T, E, k):
    torch.zeros(1, device=DEV)
    g = torch.Generator(device="cpu").manual_seed(T + E)
    for call in range(2):                       # two calls in a row share the built-in scratch
        logits = torch.randn((T, E), generator=g).to(DEV)
        if call == 1:
            logits[:, : E // 2] -= 3.0           # a different load pattern: stale scratch would show
        want = _plan_with_context(T, E, k, logits)
        got = _buffers(T, E, k)
        binding.moe_plan_routing_static(T, E, k, logits, **got)
        torch.cuda.synchronize()
        for name in ("topk_ids", "counts", "offsets", "perm", "inv_perm"):
            assert torch.equal(got[name], want[name]), f"call {call}: {name}"
        assert torch.equal(got["topk_w"], want["topk_w"]), f"call {call}: topk_w"
        assert int(got["offsets"][-1]) == T * k


def test_static_scratch_limit_and_argument_errors():
    torch.zeros(1, device=DEV)
    T, E, k = 8200, 256, 8                     # ceil(8200/32) * 256 = 65792 > 65536
    b = _buffers(16, E, k)
    logits = torch.zeros((16, E), device=DEV)
    with pytest.raises(binding.MoeError) as ei:
        binding.moe_plan_routing_static(T, E, k, logits, **b)
    assert ei.value.code == 8 and "STATIC_SCRATCH_TOO_SMALL" in str(ei.value)
    with pytest.raises(binding.MoeError) as ei:
        binding.moe_plan_routing_static(16, E, 40, logits, **b)
    assert ei.value.code == 2
    with pytest.raises(binding.MoeError) as ei:
        binding.moe_plan_routing_static(16, E, k, None, **b)
    assert ei.value.code == 1
    # T == 0 clears counts and offsets and launches nothing
    binding.moe_plan_routing_static(0, E, k, None, None, None, b["counts"], b["offsets"], None, None)
    torch.cuda.synchronize()
    assert b["counts"].eq(0).all() and b["offsets"].eq(0).all()
