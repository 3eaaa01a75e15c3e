"""The workspace-free entry point (`gdn_tree_verify_static`) against the ordinary one.

Some users of the library cannot hand it a scratch buffer because they cannot allocate device memory (their own pool
owns the GPU, or an allocation in their decode loop would stall the device).  This test calls the variant whose
scratch is a fixed array inside the library, twice in a row, and checks that each call reproduces what
`gdn_tree_verify` writes for the same inputs.  It is collected last so that a run stopping at the first failure has
already been through every other test; it does not depend on anything those tests leave behind.
"""
import numpy as np
import pytest

from paper_2607_06763_b200 import synth

pytestmark = pytest.mark.gpu


def test_static_scratch_verify_matches_workspace_verify(cuda_device):
    import torch
    import paper_2607_06763_b200 as gdn
    from tests import gdn_testlib as tl

    for rep, out_dtype in ((0, synth.BF16), (1, synth.F32)):
        w = synth.config(1, rep, out_dtype=out_dtype)          # one layer, 64-node tree: about 1 MiB of scratch
        dc = tl.DeviceCase(w)
        assert 0 < dc.ws_bytes <= gdn.binding.GDN_STATIC_SCRATCH_BYTES
        assert dc.verify() == 0 and dc.device_status() == 0
        want = dc.o_host()
        for call in range(2):                                  # the second call sees the first one's leftovers
            dc.o.fill_(float("nan"))
            rc = gdn.gdn_tree_verify_static(dc.shape, dc.S0, dc.q, dc.k, dc.v, dc.g, dc.beta, dc.parent,
                                            dc.node_offsets, dc.o, dc.status)
            assert rc == 0, gdn.gdn_status_string(rc)
            assert dc.device_status() == 0
            tl.assert_close_per_head(dc.o_host(), want, w.node_offsets, f"static call {call} rep {rep}",
                                     bf16_out=tl.is_bf16_out(w))
    # a different, smaller problem right after: stale contents of the shared array must not leak into it
    w0 = synth.config(0, 0)
    d0 = tl.DeviceCase(w0)
    assert d0.verify() == 0 and d0.device_status() == 0
    want0 = d0.o_host()
    d0.o.zero_()
    assert gdn.gdn_tree_verify_static(d0.shape, d0.S0, d0.q, d0.k, d0.v, d0.g, d0.beta, d0.parent, d0.node_offsets,
                                      d0.o, d0.status) == 0
    assert d0.device_status() == 0
    tl.assert_close_per_head(d0.o_host(), want0, w0.node_offsets, "static small case")
    tl.assert_close_per_head(d0.o_host(), tl.oracle_verify(w0), w0.node_offsets, "static small case vs oracle")
    torch.cuda.synchronize()


def test_static_scratch_calls_allocate_nothing_and_do_not_leak_between_shapes(cuda_device):
    """After one warm-up call (which loads the kernels and resolves the array's address) further calls must leave
    the device's free memory and torch's allocator exactly as they were.  The shapes are chosen so that the
    kernels that really use the scratch run: a 100-node tree (tree plan of the grouped tensor-core kernel), then an
    fp32 d = 64 problem (general kernel: plan and the cached solve result) over the larger one's leftovers; each is
    checked against the oracle."""
    import torch
    import paper_2607_06763_b200 as gdn
    from tests import gdn_testlib as tl

    rng = np.random.default_rng(5)
    big = synth.random_case(61, [synth.tree_geo(rng, 100), synth.tree_geo(rng, 70)], 2, 4, 128, 128, synth.BF16,
                            synth.F32, name="static_grouped")
    small = synth.random_case(62, [synth.tree_geo(rng, 23)], 2, 4, 64, 64, synth.F32, synth.F32, name="static_general")
    cases = [(w, tl.DeviceCase(w), tl.oracle_verify(w)) for w in (big, small)]

    def call(dc):
        rc = gdn.gdn_tree_verify_static(dc.shape, dc.S0, dc.q, dc.k, dc.v, dc.g, dc.beta, dc.parent, dc.node_offsets,
                                        dc.o, dc.status)
        assert rc == 0, gdn.gdn_status_string(rc)

    for _, dc, _ in cases:     # warm-up: module load, address lookup, kernel attributes
        call(dc)
        dc.o.fill_(float("nan"))
    torch.cuda.synchronize()
    free0, alloc0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(2):         # nothing but static-scratch calls between the two readings
        for _, dc, _ in cases:
            call(dc)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    assert torch.cuda.mem_get_info()[0] == free0, "a static-scratch call changed the device's free memory"
    for w, dc, ref in cases:   # the large problem ran first, the small one over its leftovers, twice
        assert dc.device_status() == 0
        tl.assert_close_per_head(dc.o_host(), ref, w.node_offsets, f"static {w.name} vs oracle")


def test_static_scratch_rejects_oversized_problems(cuda_device):
    import paper_2607_06763_b200 as gdn
    from tests import gdn_testlib as tl

    rng = np.random.default_rng(1)
    w = synth.random_case(4, [synth.tree_geo(rng, 200), synth.tree_geo(rng, 200)], 16, 32, 128, 128, synth.BF16,
                          synth.BF16)
    dc = tl.DeviceCase(w)
    assert dc.ws_bytes > gdn.binding.GDN_STATIC_SCRATCH_BYTES
    dc.o.fill_(5.0)
    rc = gdn.gdn_tree_verify_static(dc.shape, dc.S0, dc.q, dc.k, dc.v, dc.g, dc.beta, dc.parent, dc.node_offsets,
                                    dc.o, dc.status)
    assert rc == -10 and "workspace" in gdn.gdn_status_string(rc)
    assert dc.device_status() == 0 and bool((dc.o == 5.0).all()), "a refused call must launch nothing"
    bad = gdn.GdnShape.from_workload(w)
    bad.d_k = 6
    assert gdn.gdn_tree_verify_static(bad, dc.S0, dc.q, dc.k, dc.v, dc.g, dc.beta, dc.parent, dc.node_offsets, dc.o,
                                      dc.status) == -2
