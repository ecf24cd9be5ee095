"""thanos_prune_layer_noalloc -- the sweep for callers that cannot allocate a workspace (their
allocator owns the whole GPU, or a cudaMalloc would stall their other streams).  It must give
what thanos_prune_layer gives, call after call, although every call reuses the same built-in
scratch array.  Collected last on purpose: a run that stops at the first failure has then
already run every other test."""

import numpy as np
import pytest
import torch

import workloads as WL

pytestmark = pytest.mark.gpu

DEV = "cuda"


@pytest.fixture(scope="module")
def T():
    import paper_2504_05346_b200 as T_
    from paper_2504_05346_b200 import build as B_

    B_.build()
    T_.load_library()
    return T_


def _factor(T, b, seed):
    Xt = WL.make_activations(2048, b, "f32", "student_t4", 0.02, 0, 10.0, seed, 0, mix=0.5).to(DEV)
    H = torch.zeros((b, b), dtype=torch.float32, device=DEV)
    T.hessian_accumulate(H, Xt)
    return T.prepare_inverse(H, 0.01)


def test_noalloc_matches_prune_layer_on_consecutive_calls(T):
    # call 1: fp32 weights, unstructured; call 2 right after it: bf16 weights (which also keeps
    # its fp32 working copy in the shared scratch), 2:4 -- different shapes, same scratch array
    U1, xn1 = _factor(T, 256, seed=3)
    W1 = WL.make_weight(64, 256, "f32", seed=71).to(DEV)
    U2, xn2 = _factor(T, 128, seed=4)
    W2 = WL.make_weight(48, 128, "bf16", seed=72).to(DEV)

    a1 = T.prune_layer_noalloc(W1, U1, xn1, T.UNSTRUCTURED, p=0.5, B=64)
    a2 = T.prune_layer_noalloc(W2, U2, xn2, T.NM, n=2, m=4, B=32)
    a3 = T.prune_layer_noalloc(W1, U1, xn1, T.UNSTRUCTURED, p=0.5, B=64)  # and back again
    torch.cuda.synchronize()
    r1 = T.prune_layer(W1, U1, xn1, T.UNSTRUCTURED, p=0.5, B=64)
    r2 = T.prune_layer(W2, U2, xn2, T.NM, n=2, m=4, B=32)

    for got, ref in ((a1, r1), (a2, r2), (a3, r1)):
        assert torch.equal(got[1], ref[1])  # masks bit for bit
        g, r = got[0].double().cpu().numpy(), ref[0].double().cpu().numpy()
        assert np.linalg.norm(g - r) <= 1e-6 * np.linalg.norm(r)
        assert got[2].n_pruned == ref[2].n_pruned and got[2].status == 0
    assert a1[2].n_pruned == 64 * 256 // 2 and a2[2].n_pruned == 48 * 128 // 2


def test_noalloc_calls_leave_device_memory_untouched(T):
    """With the outputs and the statistics buffer created beforehand, a call must not change the
    amount of device memory in use: neither PyTorch's allocator nor the driver's free-memory count
    moves across three calls (after a first call that looks up the scratch address), and calls
    share no state beyond the scratch (identical statistics for identical inputs)."""
    U, xn = _factor(T, 256, seed=6)
    W = WL.make_weight(64, 256, "f32", seed=74).to(DEV)
    out = torch.empty_like(W)
    mask = torch.empty(W.shape, dtype=torch.uint8, device=DEV)
    stats = [torch.zeros(64, dtype=torch.uint8, device=DEV) for _ in range(3)]
    lib = T.load_library()
    args = lambda st: (W.data_ptr(), out.data_ptr(), mask.data_ptr(), T.F32, 64, 256, U.data_ptr(),
                       xn.data_ptr(), T.UNSTRUCTURED, 0.5, 0, 0, 64, st.data_ptr(),
                       torch.cuda.current_stream().cuda_stream)
    warm = torch.zeros(64, dtype=torch.uint8, device=DEV)
    assert lib.thanos_prune_layer_noalloc(*args(warm)) == 0      # first call: address look-up
    import gc
    gc.collect()   # leftovers of earlier tests must not be freed between the two readings
    torch.cuda.synchronize()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    free0, _ = torch.cuda.mem_get_info()
    gc.disable()
    try:
        for st in stats:
            assert lib.thanos_prune_layer_noalloc(*args(st)) == 0
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        alloc1, reserved1 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    finally:
        gc.enable()
    assert alloc1 == alloc0 and reserved1 == reserved0
    assert free1 == free0
    assert torch.equal(stats[0], stats[1]) and torch.equal(stats[1], stats[2])
    ref = T.prune_layer(W, U, xn, T.UNSTRUCTURED, p=0.5, B=64)
    assert torch.equal(mask, ref[1]) and torch.equal(out, ref[0])


def test_noalloc_refuses_layers_beyond_its_fixed_scratch(T):
    U, xn = _factor(T, 256, seed=5)
    big = torch.zeros((8192, 256), dtype=torch.float32, device=DEV)  # needs > 4 MiB of scratch
    assert T.workspace_bytes(2, 8192, 256, 128, T.F32) > 4 << 20
    with pytest.raises(T.ThanosError) as e:
        T.prune_layer_noalloc(big, U, xn, T.UNSTRUCTURED, p=0.5, B=128)
    assert e.value.code == 5  # THANOS_ERR_WORKSPACE, nothing was launched
    # a layer that fits still works afterwards
    W = WL.make_weight(32, 256, "f32", seed=73).to(DEV)
    out, mask, st = T.prune_layer_noalloc(W, U, xn, T.NM, n=2, m=4, B=64)
    assert st.n_pruned == 32 * 256 // 2
