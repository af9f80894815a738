"""moe_permute_static_scratch: the route-permute variant for callers that cannot allocate device
memory (its scratch is a fixed array inside the library).  It must give exactly what moe_permute
gives -- and what the CPU oracle gives -- call after call, although all calls share that one array,
and a call must leave the amount of free device memory as it found it.  This file sorts last so that
a run stopping at the first failure has already run everything else."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O


def _routing(T, E, K, seed):
    rng = np.random.default_rng(seed)
    idx = rng.integers(0, E, size=(T, K)).astype(np.int32)
    if E > 2:
        idx[idx == 1] = E - 1          # leave one expert without rows
    return idx


def _run(B, fn, d, x, idx, H):
    R = idx.numel()
    E = d.E
    out = dict(counts=torch.full((E,), -1, dtype=torch.int32, device="cuda"),
               offsets=torch.full((E + 1,), -1, dtype=torch.int32, device="cuda"),
               r2p=torch.full((R,), -1, dtype=torch.int32, device="cuda"),
               p2r=torch.full((R,), -1, dtype=torch.int32, device="cuda"),
               xp=torch.full((R, H), float("nan"), dtype=torch.bfloat16, device="cuda"))
    fn(out)
    torch.cuda.synchronize()
    return out


@pytest.mark.gpu
def test_static_scratch_permute_matches_moe_permute_on_consecutive_calls():
    from paper_2606_26453_b200 import binding as B
    B.load_library()
    # two calls in a row with different sizes and routings: the second must not see the first's leftovers
    for T, H, E, K, seed in ((4096, 256, 64, 6, 0), (1500, 128, 9, 4, 1), (4096, 256, 64, 6, 2)):
        d = B.dims(T, H, 128, E, K)
        idx = torch.from_numpy(_routing(T, E, K, seed)).cuda()
        x = torch.randn((T, H), device="cuda", generator=torch.Generator("cuda").manual_seed(seed)).to(torch.bfloat16)
        ws = torch.empty(max(B.moe_permute_workspace_bytes(d), 16), dtype=torch.uint8, device="cuda")
        ref = _run(B, lambda o: B.moe_permute(d, x, idx, o["xp"], o["counts"], o["offsets"], o["r2p"], o["p2r"], ws),
                   d, x, idx, H)
        for _ in range(2):
            got = _run(B, lambda o: B.moe_permute_static_scratch(d, x, idx, o["xp"], o["counts"], o["offsets"],
                                                                 o["r2p"], o["p2r"]), d, x, idx, H)
            for k in ref:                                   # integers and row copies: bit-exact
                assert torch.equal(got[k], ref[k]), (k, T, E, K)
        # and against the oracle: the stable sort itself, and bit copies of the token rows
        oc, oo, or2p, op2r = O.permute_indices(idx.cpu().numpy(), E)
        assert np.array_equal(got["counts"].cpu().numpy(), oc) and np.array_equal(got["offsets"].cpu().numpy(), oo)
        assert np.array_equal(got["r2p"].cpu().numpy(), or2p) and np.array_equal(got["p2r"].cpu().numpy(), op2r)
        assert torch.equal(got["xp"], x[torch.from_numpy(or2p.astype(np.int64) // K).cuda()])
        # what the entry point exists for: a call (after the first one on this device, which resolved the
        # array's address) allocates nothing -- the free device memory is the same before and after
        out = dict(got)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        B.moe_permute_static_scratch(d, x, idx, out["xp"], out["counts"], out["offsets"], out["r2p"], out["p2r"])
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before
    assert B.moe_device_status() == 0


def test_static_scratch_permute_rejects_sizes_beyond_its_array():
    """ceil(T*K/256)*E*4 bytes above the 4 MiB array: refused on the host, nothing launched."""
    from paper_2606_26453_b200 import binding as B, build
    build.build_library()
    lib = B.load_library()
    big = B.dims(1 << 20, 128, 128, 1024, 8)
    assert B.moe_permute_workspace_bytes(big) > (4 << 20)
    p = ctypes.c_void_p
    rc = lib.moe_permute_static_scratch(ctypes.byref(big), p(256), p(256), p(256), p(256), p(256), p(256), p(256), None)
    assert rc == 5
    assert "too small" in B.status_string(rc)
