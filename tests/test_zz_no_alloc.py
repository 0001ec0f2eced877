"""The no-allocation entry point, vig_bigla_fwd_static_bf16 (collected last on purpose).

It serves callers that may not allocate device memory at call time (fixed memory budgets, shared
GPUs under a hard partition, hosts that give the library no allocator): its scratch is a fixed
array inside the library.  The test calls it through the C ABI twice in a row on a sequence long
enough to need that scratch and checks both results against the ordinary entry point, then checks
that a problem too large for the fixed array is refused before anything is launched.
"""
import numpy as np
import pytest
import torch

import paper_2405_18425_b200 as vig
from paper_2405_18425_b200 import synth

from helpers import to_device

pytestmark = pytest.mark.gpu

STATIC_BYTES = 24 * 1024 * 1024


def _problem(seed, units, L, dk, dv):
    cfg = synth.BiglaConfig("noalloc", B=units, H=1, L=L, dk=dk, dv=dv, dtype="bf16", gate_mean=0.0, seed=seed)
    x = synth.make_inputs(cfg)
    d = {n: to_device(a, "bf16") for n, a in x.items()}
    la_f, la_b = torch.empty_like(d["g_fwd"]), torch.empty_like(d["g_bwd"])
    vig.vig_gate_prep_bf16(d["g_fwd"], d["g_bwd"], la_f, la_b, 16.0)
    return d["q"], d["k"], d["v"], la_f, la_b


def test_static_scratch_entry_matches_regular_entry_twice():
    lib = vig.load()
    args_a = _problem(11, 5, 1500, 24, 48)      # 12 segments per unit: needs the scratch
    args_b = _problem(12, 3, 777, 32, 64)       # a different shape right after, same shared scratch
    assert 0 < vig.vig_bigla_workspace_bytes(5, 1, 1500, 24, 48) <= STATIC_BYTES
    outs = {id(a): torch.full_like(a[2], float("nan")) for a in (args_a, args_b)}   # made before the free-memory readings
    for n, args in enumerate((args_a, args_b, args_a)):
        q, k, v, la_f, la_b = args
        ref = torch.full_like(v, float("nan"))
        vig.vig_bigla_fwd_bf16(q, k, v, la_f, la_b, ref)
        B, H, L, dk = q.shape
        for rep in range(2):                     # two calls in a row reuse whatever the last one left behind
            out = outs[id(args)]
            out.fill_(float("nan"))
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            st = lib.vig_bigla_fwd_static_bf16(q.data_ptr(), k.data_ptr(), v.data_ptr(), la_f.data_ptr(),
                                               la_b.data_ptr(), out.data_ptr(), B, H, L, dk, v.shape[3],
                                               torch.cuda.current_stream().cuda_stream)
            assert st == 0
            torch.cuda.synchronize()
            if n > 0 or rep > 0:                 # past the first call (one-time set-up): the device's free memory does not move
                assert torch.cuda.mem_get_info()[0] == free_before
            got, want = out.float().cpu().numpy(), ref.float().cpu().numpy()
            assert np.isfinite(got).all()
            assert np.abs(got - want).max() <= 2e-2 * np.abs(want).max()
            assert torch.equal(out.view(torch.int16), ref.view(torch.int16))   # same kernels, same order: same bits
    assert vig.vig_last_device_status() == 0


def test_static_scratch_entry_short_sequences_and_limits():
    lib = vig.load()
    q, k, v, la_f, la_b = _problem(13, 4, 196, 32, 64)   # one block per unit: the scratch is not even touched
    ref, out = torch.empty_like(v), torch.empty_like(v)
    vig.vig_bigla_fwd_bf16(q, k, v, la_f, la_b, ref)
    vig.vig_bigla_fwd_static_bf16(q, k, v, la_f, la_b, out)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), ref.view(torch.int16))
    # too large for the fixed array: refused with VIG_ERR_WORKSPACE, nothing launched, pointers never touched
    assert vig.vig_bigla_workspace_bytes(64, 4, 4096, 32, 64) > STATIC_BYTES
    before = vig.vig_kernel_launch_count()
    p = q.data_ptr()
    assert lib.vig_bigla_fwd_static_bf16(p, p, p, p, p, p, 64, 4, 4096, 32, 64, None) == -6
    assert lib.vig_bigla_fwd_static_bf16(p, p, p, p, p, p, 2, 2, 300, 40, 72, None) == -3
    assert lib.vig_bigla_fwd_static_bf16(None, p, p, p, p, p, 2, 2, 300, 32, 64, None) == -1
    assert vig.vig_kernel_launch_count() == before
