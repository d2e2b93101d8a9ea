"""Decode without a caller workspace (kvq_decode_attention_static).

Who needs it: callers that are not allowed to allocate device memory around a
decode step - a serving engine whose own arena already owns all free HBM (a
cudaMalloc there stalls the device and may simply fail), or a plug-in that gets
nothing but input/output pointers from its host.  The entry point keeps the
split partials in an 8 MiB buffer inside the library instead.

The test goes through the C-ABI, makes two calls in a row (the second on another
cache and shape, so the buffer still holds the first call's partials) and checks
each against the regular entry point (bit for bit: both run the same kernels) and one case against the
fp64 oracle; neither torch's allocator nor the driver's free-memory figure may move across a call.
This file is collected last on purpose.
"""
import gc as gc_mod

import numpy as np
import pytest
import torch

from paper_2502_15075_b200 import workloads as wl

import kvq_testlib as tl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kvq():
    from paper_2502_15075_b200 import build
    build.build()
    from paper_2502_15075_b200 import kvq as mod
    return mod


def _allocations() -> int:
    """Requests torch's caching allocator has served so far (a counter that never goes down, unlike the
    bytes in use, which drop whenever the garbage collector releases an unrelated tensor)."""
    return torch.cuda.memory_stats().get("allocation.all.allocated", 0)


def _case(kvq, w, B, T, seed):
    k, v = wl.make_kv(w, layer=seed, tokens=T, batch=B)
    cap = ((T + 127) // 128) * 128
    cfg, gc, _ = tl.build_both(kvq, w, k, v, [T], cap)
    q = wl.make_q(w, layer=seed, batch=B).cuda()
    return cfg, gc, q


def test_static_scratch_decode_matches_workspace_decode_twice(kvq):
    cases = [_case(kvq, wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8), 2, 1000, 0),
             _case(kvq, wl.LLAMA_1B.with_(n_kv_heads=4, n_q_heads=16), 3, 333, 1)]
    free_after_first = None
    for i, (cfg, gc, q) in enumerate(cases):  # two calls in a row on the shared built-in buffer
        ref = torch.from_numpy(tl.gpu_decode(kvq, cfg, gc, q))
        out = torch.full(tuple(q.shape), float("nan"), dtype=torch.float32, device="cuda")
        gc_mod.collect()     # tensors left over from earlier tests are freed now, not in the middle of the check
        torch.cuda.synchronize()
        n_alloc = _allocations()
        free0 = torch.cuda.mem_get_info()[0]
        kvq.kvq_decode_attention_static(cfg, gc, q, out)
        torch.cuda.synchronize()
        assert _allocations() == n_alloc      # torch's allocator served no request during the call
        if i > 0:            # after the first call's one-time address lookup the driver's free memory does not move
            assert torch.cuda.mem_get_info()[0] == free0
        assert kvq.kvq_check_status(gc) == 0
        # same kernels, same split plan: the two entry points agree bit for bit
        assert torch.equal(out.double().cpu(), ref)
        if i == 0:           # and one case against the fp64 oracle on the same codes
            want = tl.oracle_on_gpu_codes(gc, wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8)).decode(tl.bits_of(q))
            tl.assert_attention_close(out.double().cpu().numpy(), want)
    # and the first configuration once more, after the buffer was used by a different shape
    cfg, gc, q = cases[0]
    out = torch.empty(tuple(q.shape), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    kvq.kvq_decode_attention_static(cfg, gc, q, out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert np.array_equal(out.double().cpu().numpy(), tl.gpu_decode(kvq, cfg, gc, q))


def test_static_scratch_rejects_oversized_problem(kvq):
    # 512 sequences x 64 query heads need ~17 MB of split partials: more than the built-in 8 MiB
    cfg = kvq.make_config(512, 64, 8, 128, 4, 2, 128, 128, 0, "bf16", 128)
    assert kvq.kvq_workspace_bytes(cfg) > kvq.STATIC_SCRATCH_BYTES
    gc = kvq.Cache(cfg)
    q = torch.zeros((512, 64, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((512, 64, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(kvq.KvqError) as e:
        kvq.kvq_decode_attention_static(cfg, gc, q, out)
    assert e.value.code == -8 and "built-in" in str(e.value)
