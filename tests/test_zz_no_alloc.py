"""slim_linear_fwd_noalloc: the forward for hosts that cannot allocate device
memory (no workspace argument; scratch is the library's built-in array).

Collected last on purpose, so that a run stopping at the first failure has
already gone through every other test.  The GPU test checks the entry point
against slim_linear_fwd on the same inputs, twice in a row, because the second
call starts from whatever the first one left in the shared scratch."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_09615_b200 import binding as K, build, inputs, parity


def test_noalloc_rejects_problems_beyond_its_scratch_on_the_host():
    """Host-side checks come before any device work: a problem whose partial
    sums would not fit the built-in array is refused with SLIM_ERR_WORKSPACE,
    one the decode kernel does not take with SLIM_ERR_UNSUPPORTED_SHAPE."""
    build.build()
    lib = K.lib()
    fake = 4096          # aligned, never dereferenced: the call must fail before touching it
    too_big = lib.slim_linear_fwd_noalloc(fake, 16, fake, fake, 1.0, fake, fake, 64, 65536, 28672, fake, None, None)
    assert too_big == K.SLIM_ERR_WORKSPACE
    assert lib.slim_linear_fwd_noalloc(fake, 17, fake, fake, 1.0, None, None, 0, 512, 512, fake, None,
                                       None) == K.SLIM_ERR_UNSUPPORTED_SHAPE
    assert lib.slim_linear_fwd_noalloc(fake, 4, fake, fake, 1.0, None, None, 0, 512, 320, fake, None,
                                       None) == K.SLIM_ERR_UNSUPPORTED_SHAPE
    assert lib.slim_linear_fwd_noalloc(None, 4, fake, fake, 1.0, None, None, 0, 512, 512, fake, None,
                                       None) == K.SLIM_ERR_INVALID_ARG
    assert K.slim_noalloc_scratch_needed(16, 65536, 28672, 64) > K.NOALLOC_SCRATCH_BYTES      # the case refused above
    assert K.slim_noalloc_scratch_needed(17, 512, 512, 0) == 0 and K.slim_noalloc_scratch_needed(4, 512, 320, 0) == 0
    # every LLaMA-2 layer shape of the workload table fits the array
    for model in inputs.LLAMA2_SHAPES.values():
        for _name, d_in, d_out, _n in model:
            r = inputs.rank_for_ratio(0.2, d_in, d_out)
            assert 0 < K.slim_noalloc_scratch_needed(16, d_out, d_in, r) <= K.NOALLOC_SCRATCH_BYTES


@pytest.mark.gpu
@pytest.mark.parametrize("d_in,d_out,r,b", [(2304, 272, 112, 13), (4096, 4096, 416, 16), (1024, 256, 0, 1)])
def test_noalloc_matches_the_workspace_entry_point_twice(d_in, d_out, r, b):
    ly = inputs.make_layer(d_in, d_out, r, b, seed=4242)
    ovals, ometa = oracle.pack(ly.codes, ly.mask)
    vals, meta = K.slim_pack(torch.from_numpy(ly.codes).cuda(), torch.from_numpy(ly.mask).cuda())
    L = K.bf16_from_bits(ly.L) if r else None
    R = K.bf16_from_bits(ly.R) if r else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    y_ref = None
    for call in range(2):
        # fresh activations per call, so a stale partial sum from the previous call would show
        x_bits = inputs.make_activations(b, d_in, 4242 + call)
        X = K.bf16_from_bits(x_bits)
        want = K.slim_linear_fwd(X, vals, meta, ly.s, L, R, kernel=K.KERNEL_DECODE)
        got = torch.full((b, d_out), float("nan"), dtype=torch.bfloat16, device="cuda")
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        free_before, _total = torch.cuda.mem_get_info()     # the driver's view: sees any cudaMalloc, torch's or not
        K.slim_linear_fwd_noalloc(X, vals, meta, ly.s, L, R, got, status=status)
        assert K.slim_last_launch_count() == 1
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() <= before     # torch may free earlier temporaries, never grow
        if call > 0:                                        # (the first call may load the kernel's code)
            assert torch.cuda.mem_get_info()[0] >= free_before
        assert K.read_status(status) == 0
        res = parity.compare(inputs.bf16_bits_to_f64(K.bits_from_bf16(got)),
                             inputs.bf16_bits_to_f64(K.bits_from_bf16(want)))
        assert res["ok"], (call, res)
        # and against the definition itself
        ref = oracle.linear_fwd(x_bits, ovals, ometa, ly.s, ly.L, ly.R)
        assert parity.compare(inputs.bf16_bits_to_f64(K.bits_from_bf16(got)), ref)["ok"]
        # same kernel, same reduction order: in fact bit-identical
        assert torch.equal(got.view(torch.int16), want.view(torch.int16))
        if y_ref is not None:
            assert not torch.equal(got.view(torch.int16), y_ref)   # the second call really used new inputs
        y_ref = got.view(torch.int16).clone()
