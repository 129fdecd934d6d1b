"""amap_execute_static: the entry point for callers that may not allocate device memory
(a plug-in inside a framework that owns the GPU's memory, a serving loop that cannot
afford cudaMalloc's device-wide synchronisation).  It must produce exactly what
amap_execute produces -- and what the CPU oracle computes -- call after call, although
every call reuses one fixed descriptor table inside the library.  Collected last on
purpose (file name)."""
import numpy as np
import pytest

from oracle import oracle
from paper_2002_12798_b200 import workloads as W

pytestmark = pytest.mark.gpu

SIGNED = {1: np.int8, 2: np.int16, 4: np.int32, 8: np.int64}


def _both_ways(B, torch, chain):
    xs = W.make_inputs(chain)
    m = B.compose_chain(chain)
    es = chain.elem_size
    dev = [torch.from_numpy(np.ascontiguousarray(x).view(SIGNED[es])).cuda() for x in xs]
    ptrs = [d.data_ptr() for d in dev]
    stream = torch.cuda.current_stream().cuda_stream
    ref = torch.full((m.out_numel,), 0x11, dtype=dev[0].dtype, device="cuda")
    m.plan(device=0).execute_ptrs(ptrs, ref.data_ptr(), stream)  # the existing entry point
    out = torch.full((m.out_numel,), 0x22, dtype=dev[0].dtype, device="cuda")
    dry = m.plan(device=-1)  # a plan made without touching CUDA
    dry.execute_static_ptrs(ptrs, out.data_ptr(), stream)
    torch.cuda.synchronize()
    want = oracle.run_chain(chain, xs).reshape(-1)  # the independent opinion: pure copies, so bit for bit
    assert np.array_equal(out.cpu().numpy().view(want.dtype), want), chain.name
    return ref, out, dry, dev, stream  # dev is returned so that the inputs stay allocated


def test_static_table_matches_amap_execute_on_calls_in_a_row():
    import torch

    from paper_2002_12798_b200 import binding as B

    cfg = W.reduced_configs()
    # different maps one after the other: each call finds the previous call's descriptors in the table
    # every kernel family reads its descriptors from the fixed table here: copy, aligned / narrow / flat
    # transposes (small panels and panels beyond the default shared-memory limit) with fills, window gather,
    # element-wise gather
    cfg["flat_destination_large_panels"] = W.c2_nhwc_to_nchw(N=40, C=128, H=35, W=35)  # 78400 bytes of shared memory
    cfg["flat_source_large_panels"] = W.c2_nchw_to_nhwc(N=40, C=128, H=35, W=35)
    for name in ("c3", "c4", "c2_fwd_narrow", "c2_fwd", "c2_inv", "flat_destination_large_panels", "c4_odd",
                 "flat_source_large_panels", "c5", "c1", "c3"):
        ref, out, dry, dev, stream = _both_ways(B, torch, cfg[name])
        ptrs = [d.data_ptr() for d in dev]
        assert torch.equal(ref, out), name  # pure copies: bit-exact
        # and the same plan twice in a row into a fresh buffer
        again = torch.zeros_like(out)
        dry.execute_static_ptrs(ptrs, again.data_ptr(), stream)
        dry.execute_static_ptrs(ptrs, again.data_ptr(), stream)
        torch.cuda.synchronize()
        assert torch.equal(ref, again), name


def test_static_table_accepts_a_plan_made_for_the_current_device():
    import torch

    from paper_2002_12798_b200 import binding as B

    chain = W.reduced_configs()["c4_odd"]
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs).reshape(-1)
    m = B.compose_chain(chain)
    plan = m.plan(device=0)  # not a dry plan: it owns a table in device memory, which this entry point ignores
    dev = [torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).cuda() for x in xs]
    stream = torch.cuda.current_stream().cuda_stream
    for _ in range(2):
        out = torch.full((m.out_numel,), 0x33, dtype=torch.int16, device="cuda")
        plan.execute_static_ptrs([d.data_ptr() for d in dev], out.data_ptr(), stream)
        torch.cuda.synchronize()
        assert np.array_equal(out.cpu().numpy().view(np.uint16), want)


def test_static_table_refuses_a_plan_that_does_not_fit():
    import torch

    from paper_2002_12798_b200 import binding as B

    # 22 inputs, each padded on both axes (a copy piece plus border pieces), joined: more pieces than the table's 64 descriptors
    n_in = 22
    b = B.Builder(2)
    ids = [b.input([4, 8]) for _ in range(n_in)]
    m = b.compose(b.concat([b.pad(t, [1, 1], [1, 1]) for t in ids], 0))
    dry = m.plan(device=-1)
    assert dry.stats()["n_pieces"] > 64
    srcs = [torch.zeros(32, dtype=torch.int16, device="cuda") for _ in range(n_in)]
    out = torch.zeros(m.out_numel, dtype=torch.int16, device="cuda")
    with pytest.raises(B.AmapError) as e:
        dry.execute_static_ptrs([s.data_ptr() for s in srcs], out.data_ptr(), 0)
    assert e.value.code == -11
