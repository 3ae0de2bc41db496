"""The no-allocation decode entry point against the regular one.

delta_attn_decode_step_noalloc serves callers that cannot allocate device memory (the host
application owns the whole GPU, or cudaMalloc's implicit synchronisation is not acceptable):
its scratch is a fixed array inside the library.  It must give the result of
delta_attn_decode_step on the same inputs, and it must do so on consecutive calls, because
every call re-uses the same array and finds the previous call's contents in it.

This file is collected last on purpose, so that a run that stops at the first failure has
already been through every other test.
"""
import numpy as np
import pytest
import torch

from paper_2507_19608_b200 import workloads as WL

pytestmark = pytest.mark.gpu


def test_noalloc_decode_matches_regular_decode_on_two_consecutive_calls():
    from paper_2507_19608_b200 import binding as B
    from tests.gpu_helpers import run_prefill, to_dev

    Bn, H, Hk, T, d, dtype, theta, W, steps = 2, 8, 2, 300, 64, "bf16", 0.15, 16, 2
    w = WL.Workload("noalloc", Bn, H, Hk, T, d, dtype, 0.95, 0.5, W, (), 4242, n_decode=steps)
    t = WL.make_qkv(w)
    st, _, kc, vc = run_prefill(B, t["q"], t["k"], t["v"], theta, W, dtype, shape="sliding", T_max=T + steps)
    # the no-alloc entry runs the FP32-pipe decode kernel: make the regular entry take the same one,
    # so that the two results must be identical bit for bit
    B.delta_state_set_decode_kernel(st, 0)

    # the carried state after prefill, copied out for the stateless entry point
    qhat_a = B.delta_state_view(st, B.DELTA_VIEW_QHAT).clone()
    qhat_b = torch.empty_like(qhat_a)
    R2 = B.delta_state_view(st, B.DELTA_VIEW_R).clone()
    kc2, vc2 = kc.clone(), vc.clone()

    for s in range(steps):
        qn, kn, vn = (to_dev(t[name][:, :, s], dtype) for name in ("q_dec", "k_dec", "v_dec"))
        ref = torch.full((Bn, H, d), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.delta_attn_decode_step(st, qn, kn, vn, kc, vc, ref, theta, W)
        got = torch.full_like(ref, float("nan"))
        B.delta_attn_decode_step_noalloc(qn, kn, vn, kc2, vc2, got, qhat_a, qhat_b, R2, T + s, Bn, H, Hk, d,
                                         T + steps, dtype, theta, W)
        torch.cuda.synchronize()
        # same kernel, same inputs, same slicing: identical (which is inside any tolerance)
        assert torch.isfinite(got.float()).all()
        assert torch.equal(got, ref), f"step {s}: {(got.float() - ref.float()).abs().max().item()}"
        n = T + s
        assert torch.equal(kc2[:, :, n], kc[:, :, n]) and torch.equal(vc2[:, :, n], vc[:, :, n])
        R_ref = B.delta_state_view(st, B.DELTA_VIEW_R)
        assert torch.equal(R2[:, :, :n + 1], R_ref[:, :, :n + 1])
        assert torch.equal(qhat_b, B.delta_state_view(st, B.DELTA_VIEW_QHAT))
        qhat_a, qhat_b = qhat_b, qhat_a
    assert B.delta_noalloc_device_status() == 0          # no bounded wait ran out in either step


def test_noalloc_rejects_what_does_not_fit_its_scratch():
    from paper_2507_19608_b200 import binding as B
    x = torch.zeros(16, dtype=torch.float32, device="cuda")
    y = torch.zeros(16, dtype=torch.float32, device="cuda")
    # B * H * (d + 2) = 64 * 32 * 66 > 32768: beyond the fixed scratch, nothing may be launched
    with pytest.raises(B.DeltaError) as e:
        B.delta_attn_decode_step_noalloc(x, x, x, x, x, x, x, y, x, 10, 64, 32, 8, 64, 128, "bf16", 0.1, 4)
    assert e.value.status == B.DELTA_ERR_SCRATCH_LIMIT
    with pytest.raises(B.DeltaError) as e:
        B.delta_attn_decode_step_noalloc(x, x, x, x, x, x, x, x, x, 10, 1, 8, 2, 64, 128, "bf16", 0.1, 4)
    assert e.value.status == B.DELTA_ERR_INVALID_ARG      # qhat_in == qhat_out
    with pytest.raises(B.DeltaError) as e:                # a cache pointer off the 16-byte grid
        B.delta_attn_decode_step_noalloc(x, x, x, x.data_ptr() + 4, x, x, x, y, x, 10, 1, 8, 2, 64, 128, "bf16", 0.1, 4)
    assert e.value.status == B.DELTA_ERR_INVALID_ARG
