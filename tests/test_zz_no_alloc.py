"""cafeq_rtn_noalloc: the entry point for callers that may not allocate device memory (allocator callbacks,
code between another library's no-allocation sections, processes with a fixed memory budget).  It must give
exactly what cafeq_rtn gives, call after call, although every call reuses one built-in scratch buffer that
still holds the previous call's data.

This file is named to be collected last, so a run that stops at the first failure has already run the
rest of the suite."""
import numpy as np
import pytest

import cafeq_synth as syn
from parity_utils import f32_dev, to_dev

torch = pytest.importorskip("torch")


@pytest.mark.gpu
def test_noalloc_matches_rtn_on_two_calls_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2511_19705_b200 as cq
    cq.lib()
    # two different problems back to back: the second starts from the first one's leftovers in the scratch.
    # The first goes through the tensor-core pass (k = 128 on the input axis), the second through the
    # shape-agnostic kernels (k = 32 on the output axis, per-channel scales).
    cases = [dict(shape=(256, 512), seed=71, bits=4, group=128, k=128, axis=cq.AXIS_IN),
             dict(shape=(96, 160), seed=72, bits=3, group=0, k=32, axis=cq.AXIS_OUT),
             dict(shape=(256, 512), seed=73, bits=4, group=128, k=128, axis=cq.AXIS_IN)]
    for c in cases:
        d_out, d_in = c["shape"]
        Wd = to_dev(syn.weight_student_t(d_out, d_in, c["seed"], 2, 10.0))
        nb = (d_in if c["axis"] == cq.AXIS_IN else d_out) // c["k"]
        Td = f32_dev(syn.perturbed_blocks(nb, c["k"], c["seed"], 0.2))
        kw = dict(bits=c["bits"], group=c["group"], tblock=c["k"], taxis=c["axis"])
        ref_codes, ref_scales = cq.cafeq_rtn(Wd, Td, **kw)
        g = c["group"] or d_in
        codes = torch.full((d_out, d_in), 99, dtype=torch.int8, device="cuda")
        scales = torch.full((d_out, d_in // g), -1.0, dtype=torch.float32, device="cuda")
        before = torch.cuda.memory_allocated()
        cq.cafeq_rtn_noalloc(Wd, Td, codes, scales, **kw)
        assert torch.cuda.memory_allocated() == before            # nothing came from torch's allocator either
        torch.cuda.synchronize()
        # same kernels on the same inputs: identical integers and identical fp32 scales
        assert torch.equal(codes, ref_codes)
        assert torch.equal(scales, ref_scales)


@pytest.mark.gpu
def test_noalloc_refuses_what_does_not_fit():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2511_19705_b200 as cq
    # per-channel scales without a transform: neither the streaming kernel nor the tensor-core pass covers it, so the
    # call needs matrix-sized scratch; the limit is what cafeq_rtn_workspace_size reports for the call
    for d_out, d_in, fits in [(1024, 1536, True), (1024, 1792, False), (4096, 3584, False)]:
        need = cq.rtn_workspace_size(cq.make_desc(d_out, d_in, 3, 0), False)
        assert (need <= cq.NOALLOC_SCRATCH_BYTES) == fits, (d_out, d_in, need)
        Wd = to_dev(syn.weight_student_t(d_out, d_in, 5, 0, 1.0))
        codes = torch.zeros((d_out, d_in), dtype=torch.int8, device="cuda")
        scales = torch.zeros((d_out, 1), dtype=torch.float32, device="cuda")
        if fits:
            cq.cafeq_rtn_noalloc(Wd, None, codes, scales, bits=3, group=0)      # first call of this shape: warms up
            torch.cuda.synchronize()
            free0 = torch.cuda.mem_get_info()[0]
            cq.cafeq_rtn_noalloc(Wd, None, codes, scales, bits=3, group=0)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free0                        # the device's free memory did not move
            ref_codes, ref_scales = cq.cafeq_rtn(Wd, None, bits=3, group=0)
            assert torch.equal(codes, ref_codes) and torch.equal(scales, ref_scales)
        else:
            with pytest.raises(cq.CafeqError) as e:
                cq.cafeq_rtn_noalloc(Wd, None, codes, scales, bits=3, group=0)
            assert e.value.code == 8 and "scratch" in str(e.value)
    # grouped scales without a transform stream through one kernel and need no scratch at any size
    assert cq.rtn_workspace_size(cq.make_desc(4096, 3584, 3, 128), False) == 0
