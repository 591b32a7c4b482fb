"""``mulo_round_static``: the fused round for hosts that cannot allocate device memory
(a server whose pool already owns all of HBM, a plug-in without an allocator, a loop that
must not hit cudaMalloc's device synchronisation).  It runs on a fixed scratch array inside
the library instead of a caller-allocated workspace, so it must give exactly what
``mulo_round`` gives -- on a first call, and on a second call that finds the first call's
leftovers in the array.  Collected last on purpose: a failure here cannot hide another test.
"""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2601_05149_b200 import binding, synth

import parity_util as pu

pytestmark = pytest.mark.gpu

KEYS = ("out_tok", "reject_bits", "expand_bits", "n_reject", "n_expand", "first_reject", "p_tok", "q_tok",
        "accept_prob")


def _static_round(ctx, cfg, batch, status, **over):
    p = binding.params_from_config(cfg, **over)
    o = binding.alloc_round_outputs(p, batch["cond"].device, True)      # allocated by the test, not the call
    ctx.mulo_round_static(p, batch["cond"], batch["uncond"], batch["draft_lo"], batch["tok_lo"], batch["nn"],
                          o["out_tok"], o["reject_bits"], o["expand_bits"], o["p_tok"], o["q_tok"],
                          o["accept_prob"], o["n_reject"], o["n_expand"], o["first_reject"], status)
    torch.cuda.synchronize()
    return pu.finish_outputs(o, cfg.W)


def test_static_scratch_round_equals_workspace_round():
    assert torch.cuda.is_available()
    binding.lib()
    ref_ctx = binding.Context(0)          # the existing entry point, with a torch-allocated workspace
    ctx = binding.Context(0)              # never given a workspace
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")

    # call 1: top-k rows (the streaming kernel), CFG, four images
    big = synth.RoundConfig("na1", B=4, H=8, W=8, V=4096, dtype="bf16", sigma=1.0, cfg_scale=3.0, top_k=500,
                            radius=2, seed=301)
    b1 = pu.build_batch(big)
    want1 = pu.gpu_round(ref_ctx, big, b1)
    got1 = _static_round(ctx, big, b1, status)
    for k in KEYS:
        assert np.array_equal(got1[k], want1[k]), k
    assert int(status.item()) == 0
    assert want1["n_reject"].sum() > 0

    # call 2, straight after: fewer positions, another round index, the general kernel with
    # pooling -- the array still holds call 1's flags and candidates beyond this call's range
    small = synth.RoundConfig("na2", B=1, H=6, W=10, V=2048, r=1, dtype="f32", sigma=1.0, top_k=0, pool_k=64,
                              pool_delta=0.3, radius=1, seed=302)
    b2 = pu.build_batch(small)
    want2 = pu.gpu_round(ref_ctx, small, b2, round=3)
    got2 = _static_round(ctx, small, b2, status, round=3)
    for k in KEYS:
        assert np.array_equal(got2[k], want2[k]), k
    assert int(status.item()) == 0

    # both agree with the oracle within the tolerances of the parity tests
    pu.check_round(big, got1, pu.oracle_images(big, b1, list(range(big.B))))
    pu.check_round(small, got2, pu.oracle_images(small, b2, [0], round=3))

    # status bits are this call's own: a token outside the vocabulary is reported, and gone on the next call
    bad = dict(b2)
    bad["tok_lo"] = b2["tok_lo"].clone()
    bad["tok_lo"][0, 0, 0] = small.V + 1
    _static_round(ctx, small, bad, status)
    assert int(status.item()) & binding.DEV_BAD_TOKEN
    _static_round(ctx, small, b2, status)
    assert int(status.item()) == 0

    o_big = binding.alloc_round_outputs(binding.params_from_config(big), "cuda", False)   # before the memory reading below

    # a request beyond the array is refused before anything is launched
    huge = binding.make_params(32, 64, 64, 4096, 2, binding.BF16)
    assert binding.Context.workspace_bytes(huge) > binding.STATIC_SCRATCH_BYTES
    launches = ctx.kernel_launches()
    dummy = torch.empty(64, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.MuloError) as e:
        ctx.mulo_round_static(huge, b1["cond"], None, b1["draft_lo"], b1["tok_lo"], None, dummy, dummy, dummy)
    assert e.value.status == binding.ERR_WORKSPACE and ctx.kernel_launches() == launches

    # an invalid argument (a misaligned tensor, a missing output) is refused before anything is
    # enqueued, the clearing of the shared array's status word included
    p2 = binding.params_from_config(small)
    o = binding.alloc_round_outputs(p2, "cuda", False)
    skewed = torch.empty(b2["cond"].numel() + 4, dtype=b2["cond"].dtype, device="cuda")[1:1 + b2["cond"].numel()]
    assert skewed.data_ptr() % 16 != 0
    launches = ctx.kernel_launches()
    with pytest.raises(binding.MuloError) as e:
        ctx.mulo_round_static(p2, skewed.view(b2["cond"].shape), None, b2["draft_lo"], b2["tok_lo"], b2["nn"],
                              o["out_tok"], o["reject_bits"], o["expand_bits"])
    assert e.value.status == binding.ERR_INVALID_ARG and ctx.kernel_launches() == launches
    with pytest.raises(binding.MuloError):
        ctx.mulo_round_static(p2, b2["cond"], None, b2["draft_lo"], b2["tok_lo"], b2["nn"], None,
                              o["reject_bits"], o["expand_bits"])

    # the call allocates nothing: free device memory is the same before and after warmed-up calls
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for rnd in range(3):
        ctx.mulo_round_static(binding.params_from_config(big, round=rnd), b1["cond"], b1["uncond"], b1["draft_lo"],
                              b1["tok_lo"], b1["nn"], o_big["out_tok"], o_big["reject_bits"], o_big["expand_bits"])
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    ref_ctx.close()
    ctx.close()
