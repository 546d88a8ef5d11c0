"""The allocation-free entry point against the oracle and the regular one (collected last on purpose).

Callers that may not allocate device memory (a plug-in inside a framework's memory pool, a
real-time or capture-time path) use gformer_causal_linear_attn_noalloc, whose scratch is a fixed
array inside the library.  It must give what gformer_causal_linear_attn gives, call after call,
although every call reuses the same scratch with the previous call's leftovers in it.
"""
import pytest
import torch

import oracle
from gates import assert_parity, errors
from paper_2412_19829_b200 import binding as gf
from paper_2412_19829_b200 import synth

pytestmark = pytest.mark.gpu


def test_noalloc_matches_regular_entry_point_twice_in_a_row():
    gf.set_tuning(gf.GF_TUNE_FORCE_SIMT, 0)
    gf.set_tuning(gf.GF_TUNE_LINEAR_SPLIT, 0)
    assert gf.lib().gformer_noalloc_scratch_bytes() == 8 << 20
    for call, (B, H, N, d, seed) in enumerate([(2, 3, 2500, 128, 71), (1, 4, 3000, 64, 72)]):
        q, k, v = [t.cuda() for t in synth.qkv(B, H, N, d, "bf16", seed=seed, gain=1.0)]
        assert gf.workspace_bytes(B, H, N, d, 1, 0, gf.GF_BF16) <= 8 << 20
        ref = gf.causal_linear_attn(q, k, v)  # several sequence segments per chain: the scratch is really used
        out = torch.empty_like(q)
        # state in/out through the allocation-free call as well
        S = torch.zeros(B, H, d, d, device="cuda")
        z = torch.zeros(B, H, d, device="cuda")
        S_ref, z_ref = torch.zeros_like(S), torch.zeros_like(z)
        gf.causal_linear_attn(q, k, v, S_ref, z_ref)
        got = gf.causal_linear_attn_noalloc(q, k, v, out, S, z)
        torch.cuda.synchronize()
        f64 = lambda t: t.cpu().to(torch.float64).numpy()
        assert gf.lib().gformer_noalloc_last_device_status(None) == gf.GF_OK
        # the answer itself: the fp64 oracle on the same rounded inputs (output and final state)
        import numpy as np
        S_want, z_want = np.zeros((B, H, d, d)), np.zeros((B, H, d))
        want = oracle.causal_linear_attn(f64(q), f64(k), f64(v), S_want, z_want)  # leaves the final state in S_want, z_want
        assert_parity(f64(got), want, "bf16", f"no-alloc call {call} against the oracle")
        # (the state sums thousands of terms: the relative gate applies to it)
        assert errors(f64(S), S_want)["rel_l2"] <= 1e-2 and errors(f64(z), z_want)["rel_l2"] <= 1e-2
        # and the regular entry point, which uses a caller-owned workspace
        assert_parity(f64(got), f64(ref), "bf16", f"no-alloc call {call}")
        assert_parity(f64(S), f64(S_ref), "bf16", f"no-alloc state S, call {call}")
        assert_parity(f64(z), f64(z_ref), "bf16", f"no-alloc state z, call {call}")


def test_noalloc_rejects_problems_beyond_the_fixed_scratch():
    B, H, N, d = 1, 32, 32768, 128
    assert gf.workspace_bytes(B, H, N, d, 1, 0, gf.GF_BF16) > 8 << 20
    q = torch.zeros(1, 1, 128, 128, dtype=torch.bfloat16, device="cuda")  # never touched: rejected on the host
    rc = gf.lib().gformer_causal_linear_attn_noalloc(q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(), B, H, N,
                                                     d, 0, 0, None, None, gf.GF_BF16, gf.GF_BHND, None)
    assert rc == gf.GF_ERR_WORKSPACE
