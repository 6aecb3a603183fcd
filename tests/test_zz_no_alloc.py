"""The routing-plan entry point that allocates nothing (moe_plan_routing_static).

Some users of the library cannot call cudaMalloc where they need a routing plan (the device already belongs
to another memory pool, or their hook is not allowed to allocate), so this entry point keeps its scratch in a
fixed array inside the library instead of in a context.  The test calls it through the C ABI twice in a row,
with different inputs, and checks each result twice over: against the context-based moe_plan_routing (same
kernels, so the integer outputs must be identical and the weights equal to the last bit) and against the CPU
oracle's top-k and stable permutation (indices bit for bit, weights within 1e-6).  It also checks that the free
device memory the driver reports is the same before and after the call.  The file is one pytest collects last; it
must pass alone in a fresh process and after all other tests."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as orc
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


# (1000, 64, 4) and (4096, 256, 8): one scan segment; (8192, 8, 2): 64 chunks of few experts, the segmented scan;
# (8192, 256, 8): 256 chunks x 256 experts = exactly the 65536 entries the built-in scratch holds;
# (3000, 48, 3): a k that does not divide the 256 slots of a chunk.
@pytest.mark.parametrize("T,E,k", [(1000, 64, 4), (4096, 256, 8), (8192, 8, 2), (8192, 256, 8), (3000, 48, 3)])
def test_static_scratch_plan_matches_oracle_and_context_plan_twice(T, E, k):
    torch.zeros(1, device=DEV)
    g = torch.Generator(device="cpu").manual_seed(T + E)
    for call in range(2):                       # two calls in a row share the built-in scratch
        logits_host = torch.randn((T, E), generator=g)
        if call == 1:
            logits_host[:, : E // 2] -= 3.0      # a different load pattern: stale scratch would show
            logits_host[::7, 1] = logits_host[::7, 0]   # exact ties: the lower expert id must win on both sides
        logits = logits_host.to(DEV)
        want = _plan_with_context(T, E, k, logits)
        got = _buffers(T, E, k)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        reserved_before = torch.cuda.memory_reserved()
        binding.moe_plan_routing_static(T, E, k, logits, **got)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        if call == 1:     # the first call of a process may load the library's kernels; the second may not allocate
            assert free_after == free_before, "device memory changed across a call that must not allocate"
            assert torch.cuda.memory_reserved() == reserved_before
        for name in ("topk_ids", "counts", "offsets", "perm", "inv_perm"):
            assert torch.equal(got[name], want[name]), f"call {call}: {name} differs from moe_plan_routing"
        assert torch.equal(got["topk_w"], want["topk_w"]), f"call {call}: topk_w"
        # the oracle, directly
        ids, w = orc.topk_route(logits_host.numpy(), k)
        counts, offsets, perm, inv_perm = orc.plan_permutation(ids, E)
        ref = dict(topk_ids=ids.reshape(-1), counts=counts, offsets=offsets, perm=perm, inv_perm=inv_perm)
        for name, exp in ref.items():
            assert np.array_equal(got[name].cpu().numpy(), exp), f"call {call}: {name} differs from the oracle"
        assert np.abs(got["topk_w"].cpu().numpy().astype(np.float64) - w.reshape(-1)).max() <= 1e-6
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
