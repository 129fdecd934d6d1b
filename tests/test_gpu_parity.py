"""Parity of the CUDA path with the CPU oracle, bit for bit, through the C ABI."""
import os

import numpy as np
import pytest

from oracle import oracle
from paper_2002_12798_b200 import workloads as W
from chain_gen import random_chain

pytestmark = pytest.mark.gpu

SIGNED = {1: np.int8, 2: np.int16, 4: np.int32, 8: np.int64}
CANARY = 64  # elements of guard band on both sides of the output


@pytest.fixture(scope="module")
def B():
    from paper_2002_12798_b200 import binding

    return binding


def run_gpu(B, chain, xs, force=0, align=16, compose_flags=0):
    """compose -> plan -> execute on cuda:0; returns the output as a flat numpy array of raw bits."""
    import torch

    m = B.compose_chain(chain, compose_flags)
    plan = m.plan(device=0, force_kernel=force, pointer_align=align)
    es = chain.elem_size
    dev = [torch.from_numpy(np.ascontiguousarray(x).view(SIGNED[es])).cuda() for x in xs]
    band = torch.full(((m.out_numel + 2 * CANARY) * es,), 0x5A, dtype=torch.uint8, device="cuda")
    out = band[CANARY * es : (CANARY + m.out_numel) * es]
    assert out.data_ptr() % 16 == 0 or align < 16
    plan.execute_ptrs([d.data_ptr() for d in dev], out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    host = band.cpu().numpy()
    assert (host[: CANARY * es] == 0x5A).all() and (host[(CANARY + m.out_numel) * es :] == 0x5A).all(), "wrote outside the output"
    return host[CANARY * es : (CANARY + m.out_numel) * es].view(xs[0].dtype), plan


@pytest.mark.parametrize("force", [0, 1, 2], ids=["auto", "gather", "copy"])
@pytest.mark.parametrize("name", sorted(W.reduced_configs()))
def test_reduced_configs_bit_exact(B, name, force):
    chain = W.reduced_configs()[name]
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs)
    got, _ = run_gpu(B, chain, xs, force=force)
    assert np.array_equal(got, want.reshape(-1))


@pytest.mark.parametrize("name", ["c1", "c2_fwd", "c3_odd", "c4_odd", "c5_odd"])
def test_index_tagged_inputs(B, name):
    """With inputs that hold their own index the output IS the composed source-index map."""
    chain = W.reduced_configs()[name]
    for part in (0, 1):
        xs = W.make_index_tagged_inputs(chain, part)
        want = oracle.run_chain(chain, xs)
        got, _ = run_gpu(B, chain, xs)
        assert np.array_equal(got, want.reshape(-1))


def test_c1_closed_form_on_the_gpu(B):
    chain = W.c1_small_chain()
    got, _ = run_gpu(B, chain, W.make_index_tagged_inputs(chain))
    a, j, k = np.meshgrid(np.arange(64), np.arange(8), np.arange(6), indexing="ij")
    want = np.zeros((64, 48), dtype=np.int64)
    want[a, 6 * j + k] = 1024 * j + 128 * k + 128 + 2 * a
    assert np.array_equal(got.astype(np.int64).reshape(64, 48), want)


def test_random_tiny_chains(B):
    r = np.random.default_rng(20021279)
    done = 0
    for trial in range(120):
        chain = random_chain(r)
        xs = [x + np.uint32(1) for x in W.make_index_tagged_inputs(chain)]
        try:
            B.compose_chain(chain)
        except B.AmapError as e:
            assert e.code == -9
            continue
        want = oracle.run_chain(chain, xs)
        for force in (0, 1, 2):
            got, _ = run_gpu(B, chain, xs, force=force)
            assert np.array_equal(got, want.reshape(-1)), (trial, force, chain.ops)
        done += 1
    assert done >= 60


@pytest.mark.parametrize("name", ["c1", "c2_fwd_rag", "c3_odd", "c4", "c4_odd", "c5"])
def test_unfused_chain_gives_the_same_bytes(B, name):
    """One stage and one temporary per operator (the chain before data-movement elimination)."""
    chain = W.reduced_configs()[name]
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs)
    got, plan = run_gpu(B, chain, xs, compose_flags=B.COMPOSE_NO_FUSE)
    assert plan.stats()["n_stages"] == len(chain.ops)
    assert np.array_equal(got, want.reshape(-1))


def test_pairs_that_cannot_be_eliminated_become_temporaries(B):
    chain = W.Chain(
        name="awkward", dtype="bf16", inputs=[[40, 24]],
        ops=[
            {"kind": "transpose", "src": 0, "perm": [1, 0]},
            {"kind": "reshape", "src": 1, "shape": [64, 15]},
            {"kind": "transpose", "src": 2, "perm": [1, 0]},
            {"kind": "reshape", "src": 3, "shape": [24, 40]},
            {"kind": "transpose", "src": 4, "perm": [1, 0]},
            {"kind": "pad", "src": 5, "lo": [1, 0], "hi": [0, 2]},
        ],
        values="normal",
    )
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs)
    got, plan = run_gpu(B, chain, xs)
    assert plan.stats()["n_stages"] >= 2  # two reshapes that do not line up with the transposes around them
    assert np.array_equal(got, want.reshape(-1))


def test_tile_broadcast(B):
    chain = W.Chain(
        name="tile", dtype="fp16", inputs=[[3, 40]],
        ops=[{"kind": "tile", "src": 0, "reps": [5, 2]}, {"kind": "transpose", "src": 1, "perm": [1, 0]}],
        values="uniform_pm1",
    )
    xs = W.make_inputs(chain)
    got, _ = run_gpu(B, chain, xs)
    assert np.array_equal(got.reshape(80, 15), np.tile(xs[0], (5, 2)).T)


def test_repeat_upsamples(B):
    """Nearest-neighbour 2x upsampling of NHWC activations: repeat on H, then on W, one composed copy."""
    chain = W.upsample_nhwc(N=2, H=9, W=7, C=40, factor=2)
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs)
    for force in (0, 1):
        got, plan = run_gpu(B, chain, xs, force=force)
        assert plan.stats()["n_stages"] == 1
        assert np.array_equal(got, want.reshape(-1))
    assert np.array_equal(want, np.repeat(np.repeat(xs[0], 2, axis=1), 2, axis=2))


def test_split_parts_each_compose_to_one_copy(B):
    """A fused QKV projection output cut into q, k, v, each moved to [B, heads, S, D]: one plan per part."""
    for part in range(3):
        chain = W.qkv_split(B=2, S=24, heads=3, D=16, part=part)
        xs = W.make_inputs(chain)
        want = oracle.run_chain(chain, xs)
        got, plan = run_gpu(B, chain, xs)
        assert plan.stats()["n_stages"] == 1 and plan.stats()["n_launches"] == 1
        assert np.array_equal(got, want.reshape(-1))
        x = xs[0].reshape(2, 24, 3, 3, 16)  # [B, S, part, heads, D]
        assert np.array_equal(want, x[:, :, part].transpose(0, 2, 1, 3))


def test_split_into_three_outputs_is_one_launch(B):
    """q, k and v cut out of one fused projection and moved to [B, heads, S, D]: ONE composed map with three
    outputs, one plan, one kernel launch (amap_compose_multi / amap_execute_multi)."""
    import torch

    Bt, S, heads, D = 2, 40, 3, 16
    hd = heads * D
    ops = []
    for part in range(3):
        base = 1 + len(ops)
        ops.append({"kind": "split", "src": 0, "axis": 2, "sizes": [hd, hd, hd], "part": part})
        ops.append({"kind": "reshape", "src": base, "shape": [Bt, S, heads, D]})
        ops.append({"kind": "transpose", "src": base + 1, "perm": [0, 2, 1, 3]})
    chain = W.Chain(name="qkv", dtype="bf16", inputs=[[Bt, S, 3 * hd]], ops=ops, values="normal")
    outs = [3, 6, 9]
    xs = W.make_inputs(chain)
    tensors = oracle.run_chain(chain, xs, keep_intermediates=True)
    m = B.compose_chain(chain, outputs=outs)
    plan = m.plan(0)
    assert plan.stats()["n_launches"] == 1 and plan.stats()["n_stages"] == 1
    src = torch.from_numpy(xs[0].view(np.int16)).cuda()
    bands = [torch.full((n + 2 * CANARY,), 0x5A5A, dtype=torch.int16, device="cuda") for n in m.out_numels]
    dsts = [b[CANARY : CANARY + n] for b, n in zip(bands, m.out_numels)]
    plan.execute_multi_ptrs([src.data_ptr()], [d.data_ptr() for d in dsts], torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    for k, t in enumerate(outs):
        host = bands[k].cpu().numpy().view(np.uint16)
        assert (host[:CANARY] == 0x5A5A).all() and (host[-CANARY:] == 0x5A5A).all()
        assert np.array_equal(host[CANARY:-CANARY], tensors[t].reshape(-1)), k
    # the single-output entry point refuses this plan; overlapping outputs are refused as well
    with pytest.raises(B.AmapError) as e:
        plan.execute_ptrs([src.data_ptr()], dsts[0].data_ptr(), 0)
    assert e.value.code == -1
    with pytest.raises(B.AmapError) as e:
        plan.execute_multi_ptrs([src.data_ptr()], [dsts[0].data_ptr(), dsts[0].data_ptr() + 32, dsts[2].data_ptr()], 0)
    assert e.value.code == -1


def test_outputs_of_different_kernel_families_and_a_tensor_read_again(B):
    """Three results of one chain: a transposed tensor (tiled transpose kernel), its padded copy (transpose plus
    fills) and a strided slice of it (gather): each output written by its own pieces, every family indexing its
    own destination."""
    import torch

    chain = W.Chain(
        name="three", dtype="bf16", inputs=[[2, 72, 16, 24]],
        ops=[
            {"kind": "transpose", "src": 0, "perm": [0, 2, 3, 1]},                                   # 1: NHWC
            {"kind": "pad", "src": 1, "lo": [0, 1, 1, 0], "hi": [0, 1, 1, 0]},                        # 2
            {"kind": "slice", "src": 1, "start": [0, 0, 1, 0], "stop": [2, 16, 24, 72], "step": [1, 2, 3, 1]},  # 3
        ],
        values="normal",
    )
    xs = W.make_inputs(chain)
    tensors = oracle.run_chain(chain, xs, keep_intermediates=True)
    outs = [1, 2, 3]
    m = B.compose_chain(chain, outputs=outs)
    plan = m.plan(0)
    src = torch.from_numpy(xs[0].view(np.int16)).cuda()
    dsts = [torch.full((n,), 0x1111, dtype=torch.int16, device="cuda") for n in m.out_numels]
    plan.execute_multi_ptrs([src.data_ptr()], [d.data_ptr() for d in dsts], torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    for k, t in enumerate(outs):
        assert np.array_equal(dsts[k].cpu().numpy().view(np.uint16), tensors[t].reshape(-1)), k


def test_chain_cut_at_an_operator_that_is_not_a_layout_operator(B):
    """Layout operators on both sides of a compute operator (here: torch adds 1 to every element): the part before
    it is one composed copy into the operator's input, the part behind it one composed copy of its result."""
    import torch

    b = B.Builder(2)
    x = b.input([6, 64, 10])
    t = b.transpose(x, [2, 0, 1])                                # [10, 6, 64]
    o = b.opaque([t], [10, 6, 64])
    z = b.transpose(b.pad(b.reshape(o, [10, 6, 8, 8]), [0, 0, 1, 0], [0, 0, 0, 0]), [1, 0, 3, 2])  # [6, 10, 8, 9]
    first, second = b.compose_multi([t]), b.compose(z)
    xv = W.make_values(6 * 64 * 10, "bf16", "normal", np.random.default_rng(7)).reshape(6, 64, 10)
    xd = torch.from_numpy(xv.view(np.int16)).cuda()
    td = torch.zeros(first.out_numel, dtype=torch.int16, device="cuda")
    first.plan(0).execute([xd], td)
    od = td + 1                                                    # the compute operator, on the same stream
    zd = torch.zeros(second.out_numel, dtype=torch.int16, device="cuda")
    second.plan(0).execute([xd, od], zd)
    torch.cuda.synchronize()
    # the oracle: chain, operator (numpy), chain
    c1 = W.Chain(name="a", dtype="bf16", inputs=[[6, 64, 10]], ops=[{"kind": "transpose", "src": 0, "perm": [2, 0, 1]}])
    tv = oracle.run_chain(c1, [xv])
    ov = (tv.view(np.int16) + np.int16(1)).view(np.uint16)
    c2 = W.Chain(name="b", dtype="bf16", inputs=[[10, 6, 64]], ops=[
        {"kind": "reshape", "src": 0, "shape": [10, 6, 8, 8]},
        {"kind": "pad", "src": 1, "lo": [0, 0, 1, 0], "hi": [0, 0, 0, 0]},
        {"kind": "transpose", "src": 2, "perm": [1, 0, 3, 2]},
    ])
    want = oracle.run_chain(c2, [ov])
    assert np.array_equal(zd.cpu().numpy().view(np.uint16), want.reshape(-1))


@pytest.mark.parametrize("name,rows", [("c5", None), ("c5_odd", None), ("c3", 2 * 3 * 100), ("c4_odd", 3 * 9 * 11), ("c1", 64),
                                       ("c2_inv_odd_u8", 2 * 64), ("c2_fwd_f32", 2 * 13 * 12)])
def test_consumer_reads_through_the_map(B, name, rows):
    """amap_consume_row_sums: the row sums of the chain's result, computed from the inputs through the composed map
    (the result is never written), against the sums of the oracle's result."""
    import torch

    chain = W.reduced_configs()[name]
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs)
    rows = rows or want.shape[0]
    cols = want.size // rows
    m = B.compose_chain(chain)
    es = chain.elem_size
    dev = [torch.from_numpy(np.ascontiguousarray(x).view(SIGNED[es])).cuda() for x in xs]
    sums = torch.full((rows,), -1, dtype=torch.int32, device="cuda")
    m.consume_row_sums(dev, rows, cols, sums)
    torch.cuda.synchronize()
    want_sums = want.reshape(rows, cols).astype(np.uint64).sum(axis=1).astype(np.uint32)
    assert np.array_equal(sums.cpu().numpy().view(np.uint32), want_sums)


def test_quasi_affine_pieces_bit_exact(B):
    """Reshapes whose factors do not line up with the transposes around them: one quasi-affine piece (digits by
    multiply-and-shift division inside the affine kernel) instead of a temporary -- with 16-byte units where runs
    survive, element by element where forced, with guards and a further reader behind it."""
    from test_compose import _run_preserving_chain, _scattered_chain

    runs = _run_preserving_chain()
    xs = W.make_inputs(runs)
    want = oracle.run_chain(runs, xs)
    got, plan = run_gpu(B, runs, xs)
    assert plan.stats()["n_stages"] == 1 and plan.stats()["kernels"]["copy"] == 1
    assert np.array_equal(got, want.reshape(-1))
    got, plan = run_gpu(B, runs, xs, compose_flags=B.COMPOSE_NO_QUASI_AFFINE)  # the two-pass form of the same chain
    assert plan.stats()["n_stages"] == 2 and np.array_equal(got, want.reshape(-1))

    scattered = _scattered_chain()
    xs = W.make_inputs(scattered)
    want = oracle.run_chain(scattered, xs)
    got, plan = run_gpu(B, scattered, xs, compose_flags=B.COMPOSE_QUASI_AFFINE)
    assert plan.stats()["n_stages"] == 1 and plan.stats()["kernels"]["gather"] == 1
    assert np.array_equal(got, want.reshape(-1))

    guarded = _run_preserving_chain(dtype="fp32")
    guarded.ops += [
        {"kind": "pad", "src": 3, "lo": [1, 0, 0], "hi": [0, 2, 0]},
        {"kind": "slice", "src": 4, "start": [0, 1, 0], "stop": [91, 90, 8], "step": [3, 2, 1]},
    ]
    guarded.values = "raw"
    xs = [x + np.uint32(1) for x in W.make_index_tagged_inputs(guarded)]
    want = oracle.run_chain(guarded, xs)
    for flags in (0, B.COMPOSE_QUASI_AFFINE):
        got, plan = run_gpu(B, guarded, xs, compose_flags=flags)
        assert plan.stats()["n_stages"] == 1 and np.array_equal(got, want.reshape(-1))


def test_random_chains_with_quasi_affine_pieces(B):
    r = np.random.default_rng(1279800)
    quasi = 0
    for trial in range(120):
        chain = random_chain(r)
        xs = [x + np.uint32(1) for x in W.make_index_tagged_inputs(chain)]
        try:
            m = B.compose_chain(chain, B.COMPOSE_QUASI_AFFINE)
        except B.AmapError as e:
            assert e.code == -9
            continue
        quasi += any(p["quasi"] for p in m.pieces())
        want = oracle.run_chain(chain, xs)
        for force in (0, 1):
            got, _ = run_gpu(B, chain, xs, force=force, compose_flags=B.COMPOSE_QUASI_AFFINE)
            assert np.array_equal(got, want.reshape(-1)), (trial, force, chain.ops)
    assert quasi >= 4


@pytest.mark.parametrize("rows,cols,dtype", [(64, 256, "bf16"), (128, 384, "bf16"), (40, 72, "bf16"), (32, 132, "fp32"),
                                             (56, 28, "bf16"), (24, 40, "u8")])
def test_transposes_with_negative_source_strides(B, rows, cols, dtype):
    """Y[j, i] = X[rows - 1 - i, j] and Y[j, i] = X[i, cols - 1 - j] as raw statements: the tiled transpose kernels
    walk the source backwards along one index (offsets stay relative to the tensor's first byte, so 32-bit
    arithmetic wraps around harmlessly)."""
    for load_C, load_b in (([[0, -1], [1, 0]], [rows - 1, 0]), ([[0, 1], [-1, 0]], [0, cols - 1])):
        chain = W.Chain(
            name="flip_transpose", dtype=dtype, inputs=[[rows, cols]],
            ops=[{"kind": "stmts", "shape": [cols, rows],
                  "stmts": [{"bounds": [cols, rows], "load": (0, load_C, load_b), "store": ([[1, 0], [0, 1]], [0, 0])}]}],
            values="raw" if dtype == "u8" else "normal",
        )
        xs = W.make_inputs(chain)
        want = oracle.run_chain(chain, xs)
        ref = xs[0][::-1, :].T if load_b[0] else xs[0][:, ::-1].T
        assert np.array_equal(want, ref)
        got, plan = run_gpu(B, chain, xs)
        assert np.array_equal(got, want.reshape(-1)), (rows, cols, dtype, load_b)


def test_dag_with_a_shared_intermediate(B):
    """One transposed tensor feeds a slice and a pad that are joined again: two readers of one intermediate."""
    chain = W.Chain(
        name="dag", dtype="bf16", inputs=[[48, 200]],
        ops=[
            {"kind": "transpose", "src": 0, "perm": [1, 0]},                                           # 1: [200, 48]
            {"kind": "slice", "src": 1, "start": [0, 0], "stop": [200, 32], "step": [1, 2]},           # 2: [200, 16]
            {"kind": "pad", "src": 1, "lo": [0, 0], "hi": [0, 16]},                                    # 3: [200, 64]
            {"kind": "concat", "srcs": [2, 3, 2], "axis": 1},                                          # 4: [200, 96]
        ],
        values="normal",
    )
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs)
    got, plan = run_gpu(B, chain, xs)
    assert plan.stats()["n_stages"] == 1
    assert np.array_equal(got, want.reshape(-1))


def test_random_statement_chains(B):
    """Raw load/store statements with arbitrary small affine maps (interleaved and merged stores, guards,
    temporaries where a pair cannot be eliminated)."""
    from test_compose_fuzz import random_stmt_chain

    r = np.random.default_rng(2002)
    staged = 0
    for trial in range(150):
        chain = random_stmt_chain(r)
        xs = [x + np.uint32(100) for x in W.make_index_tagged_inputs(chain)]
        want = oracle.run_chain(chain, xs)
        got, plan = run_gpu(B, chain, xs, force=trial % 3)
        staged += plan.stats()["n_stages"] > 1
        assert np.array_equal(got, want.reshape(-1)), (trial, chain.ops)
    assert staged > 0


def test_offsets_beyond_4_gib(B):
    """A 5 GiB byte tensor: the pieces' source offsets do not fit 32 bits, so the 64-bit kernel variants run
    (strip kernel for the slice, transpose kernel for the slice + transpose).  Only a slab near the end is
    filled and read; the oracle sees a host array of the same shape whose untouched pages are never allocated."""
    import torch

    shape = [5, 32768, 32768]
    lo_row, rows = 100, 64
    slab = np.random.default_rng(5).integers(1, 255, size=(rows, shape[2]), dtype=np.uint8)
    host = np.zeros(shape, dtype=np.uint8)  # lazily mapped
    host[4, lo_row : lo_row + rows] = slab
    dev = torch.zeros(shape, dtype=torch.uint8, device="cuda")
    dev[4, lo_row : lo_row + rows] = torch.from_numpy(slab).cuda()
    sl = {"kind": "slice", "src": 0, "start": [4, lo_row, 0], "stop": [5, lo_row + rows, shape[2]], "step": [1, 1, 1]}
    for ops, kernel in (([sl], "copy"), ([sl, {"kind": "transpose", "src": 1, "perm": [0, 2, 1]}], "transpose")):
        chain = W.Chain(name="big", dtype="u8", inputs=[shape], ops=ops, values="raw")
        want = oracle.run_chain(chain, [host])
        m = B.compose_chain(chain)
        plan = m.plan(0)
        assert plan.stats()["kernels"][kernel] == 1
        out = torch.zeros(m.out_numel, dtype=torch.uint8, device="cuda")
        plan.execute([dev], out)
        torch.cuda.synchronize()
        assert np.array_equal(out.cpu().numpy(), want.reshape(-1)), kernel
    del dev


def test_launch_with_more_pieces_than_fit_the_kernel_parameters(B):
    """Twenty operands joined and transposed: twenty pieces in one launch, so the kernels read their descriptors
    from the plan's table in device memory instead of the kernel parameters."""
    n_in = 20
    chain = W.Chain(
        name="wide_concat", dtype="bf16", inputs=[[2, 16, 8, 8]] * n_in,
        ops=[{"kind": "concat", "srcs": list(range(n_in)), "axis": 1}, {"kind": "transpose", "src": n_in, "perm": [0, 2, 3, 1]}],
        values="normal",
    )
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs)
    got, plan = run_gpu(B, chain, xs)
    assert plan.stats()["n_pieces"] == n_in and plan.stats()["n_launches"] == 1
    assert np.array_equal(got, want.reshape(-1))


def test_random_layout_changes_on_every_transpose_kernel(B):
    """Seeded random NCHW <-> NHWC shapes (odd and even maps, channel counts around the kernels' thresholds, 2- and
    4-byte elements): whichever transpose kernel the planner picks, the bytes are the oracle's; every kernel of the
    family is met at least once."""
    rng = np.random.default_rng(12798)
    seen = {}
    for _ in range(70):
        es = int(rng.choice([2, 2, 2, 4]))
        n, h, w = int(rng.integers(1, 25)), int(rng.integers(1, 40)), int(rng.integers(1, 40))
        c = int(rng.choice([8, 16, 24, 32, 40, 48, 64, 72, 96, 128, 136, 200, 256])) if rng.random() < 0.8 else int(rng.integers(1, 200))
        n = max(1, min(n, 400_000 // (h * w * c)))
        fwd = bool(rng.random() < 0.5)
        chain = W.Chain(
            name="layout", dtype="bf16" if es == 2 else "fp32", inputs=[[n, c, h, w] if fwd else [n, h, w, c]],
            ops=[{"kind": "transpose", "src": 0, "perm": [0, 2, 3, 1] if fwd else [0, 3, 1, 2]}], values="normal",
            seed=int(rng.integers(1 << 30)),
        )
        xs = W.make_inputs(chain)
        want = oracle.run_chain(chain, xs)
        got, plan = run_gpu(B, chain, xs)
        for launch in plan.launches():
            seen[launch["kernel"]] = seen.get(launch["kernel"], 0) + 1
        assert np.array_equal(got.view(SIGNED[es]), np.ascontiguousarray(want).reshape(-1).view(SIGNED[es])), (chain.inputs, fwd)
    for kernel in ("transpose", "transpose_flat", "transpose_flat_source", "transpose_shifted", "transpose_realign"):
        assert seen.get(kernel, 0) > 0, seen


def test_flat_destination_transposes_from_the_descriptor_table(B):
    """Twenty NHWC operands joined along the batch and taken to NCHW (7x7 maps: rows of 98 bytes): twenty pieces
    of the flat-destination transpose in one launch, their descriptors read from the plan's table."""
    n_in = 20
    chain = W.Chain(
        name="wide_concat_flat", dtype="bf16", inputs=[[2, 7, 7, 72]] * n_in,
        ops=[{"kind": "concat", "srcs": list(range(n_in)), "axis": 0}, {"kind": "transpose", "src": n_in, "perm": [0, 3, 1, 2]}],
        values="normal",
    )
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs)
    got, plan = run_gpu(B, chain, xs)
    launches = plan.launches()
    assert len(launches) == 1 and launches[0]["kernel"] == "transpose_flat" and launches[0]["n_descriptors"] == n_in
    assert np.array_equal(got, want.reshape(-1))


def test_three_guards_in_one_piece(B):
    """A 3-D window gather written as one raw guarded statement: three guards, so the kernels' larger
    constraint variant runs."""
    D, H, Wd = 6, 7, 9
    chain = W.Chain(
        name="stencil", dtype="fp32", inputs=[[D, H, Wd]],
        ops=[{
            "kind": "stmts", "shape": [D * H * Wd, 27],
            "stmts": [{
                "bounds": [D, H, Wd, 3, 3, 3],
                "load": (0, [[1, 0, 0, 1, 0, 0], [0, 1, 0, 0, 1, 0], [0, 0, 1, 0, 0, 1]], [-1, -1, -1]),
                "store": ([[H * Wd, Wd, 1, 0, 0, 0], [0, 0, 0, 9, 3, 1]], [0, 0]),
                "guarded": True, "fill": 0,
            }],
        }],
        values="raw",
    )
    xs = [x + np.uint32(1) for x in W.make_index_tagged_inputs(chain)]
    want = oracle.run_chain(chain, xs)
    assert len(B.compose_chain(chain).pieces()[0]["guards"]) == 3
    for force in (0, 1):
        got, _ = run_gpu(B, chain, xs, force=force)
        assert np.array_equal(got, want.reshape(-1))


def test_sixteen_byte_elements_against_torch(B):
    """elem_size 16 (complex128): every element is a whole 16-byte unit.  Checked against torch's own permute
    (a library routine as third opinion; the oracle's Python front end stops at 8-byte elements)."""
    import torch

    x = torch.randn(3, 10, 7, dtype=torch.complex128, device="cuda")
    b = B.Builder(16)
    t = b.input([3, 10, 7])
    m = b.compose(b.pad(b.transpose(t, [2, 0, 1]), [1, 0, 0], [0, 0, 2]))
    out = torch.full((8, 3, 12), 7 + 7j, dtype=torch.complex128, device="cuda")
    m.plan(0).execute([x], out)
    torch.cuda.synchronize()
    want = torch.nn.functional.pad(x.permute(2, 0, 1), (0, 2, 0, 0, 1, 0))
    assert torch.equal(out.view(torch.int64), want.contiguous().view(torch.int64))


@pytest.mark.parametrize("dtype,es", [("u8", 1), ("u64", 8)])
def test_other_element_sizes(B, dtype, es):
    chain = W.c3_head_split(B=2, S=20, heads=3, D=16, keep=11, dtype=dtype)
    chain.values = "raw"
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs)
    got, _ = run_gpu(B, chain, xs)
    assert np.array_equal(got, want.reshape(-1))


@pytest.mark.parametrize("name", ["c4_odd", "c2_fwd_mid", "c3", "c4", "c5", "c1"])
def test_execute_host_matches(B, name):
    """Host buffers in, host buffers out.  Maps with an outer batch loop go slab by slab on extra streams
    (c2, c3, c4); the others (guards, no batch loop) in one piece."""
    import torch

    chain = W.reduced_configs()[name]
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs)
    m = B.compose_chain(chain)
    plan = m.plan(0)
    out = np.empty(m.out_numel, dtype=xs[0].dtype)
    plan.execute_host([np.ascontiguousarray(x) for x in xs], out)
    assert np.array_equal(out, want.reshape(-1))
    # pinned buffers (truly asynchronous copies), staging reused, a non-default stream
    es = chain.elem_size
    pins = [torch.from_numpy(np.ascontiguousarray(x).view(SIGNED[es])).pin_memory() for x in xs]
    pout = torch.zeros(m.out_numel, dtype=pins[0].dtype).pin_memory()
    stream = torch.cuda.Stream()
    for _ in range(2):
        pout.zero_()
        plan.execute_host(pins, pout, stream.cuda_stream)
        assert np.array_equal(pout.numpy().view(xs[0].dtype), want.reshape(-1))


def test_misaligned_pointer_is_refused(B):
    import torch

    chain = W.reduced_configs()["c3"]
    m = B.compose_chain(chain)
    plan = m.plan(0, pointer_align=16)
    buf = torch.zeros(m.out_numel * 2 + 64, dtype=torch.uint8, device="cuda")
    srcs = [torch.zeros(n * 2, dtype=torch.uint8, device="cuda") for n in m.in_numel]
    with pytest.raises(B.AmapError) as e:
        plan.execute_ptrs([s.data_ptr() for s in srcs], buf.data_ptr() + 2, 0)
    assert e.value.code == -7
    # a plan that promises only element alignment accepts it and still copies exactly
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs)
    plan2 = m.plan(0, pointer_align=2)
    dev = [torch.from_numpy(x.view(np.int16)).cuda() for x in xs]
    plan2.execute_ptrs([d.data_ptr() for d in dev], buf.data_ptr() + 2, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    got = buf.cpu().numpy()[2 : 2 + m.out_numel * 2].view(np.uint16)
    assert np.array_equal(got, want.reshape(-1))


def test_overlapping_buffers_are_refused(B):
    import torch

    chain = W.reduced_configs()["c2_fwd_rag"]
    m = B.compose_chain(chain)
    plan = m.plan(0)
    buf = torch.zeros(m.out_numel * 2 + 64, dtype=torch.int16, device="cuda")
    with pytest.raises(B.AmapError) as e:  # output starts inside the input
        plan.execute_ptrs([buf.data_ptr()], buf.data_ptr() + 32, 0)
    assert e.value.code == -1


@pytest.mark.parametrize("chain", [
    W.reduced_configs()["c2_fwd_mid"],
    W.c2_nhwc_to_nchw(N=40, C=128, H=35, W=35),  # flat-destination transpose, panels of 78400 bytes of shared memory
    W.c2_nchw_to_nhwc(N=40, C=128, H=35, W=35),  # flat-source transpose
], ids=["aligned", "flat_destination", "flat_source"])
def test_execute_can_be_captured_in_a_cuda_graph(B, chain):
    """amap_execute neither synchronises nor allocates, so a stream capture can record it; replays must copy."""
    import torch

    (x,) = W.make_inputs(chain)
    want = oracle.run_chain(chain, [x]).reshape(-1)
    m = B.compose_chain(chain)
    plan = m.plan(0)
    src = torch.from_numpy(x.view(np.int16)).cuda()
    dst = torch.zeros(m.out_numel, dtype=torch.int16, device="cuda")
    plan.execute([src], dst)  # first use outside the capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        plan.execute([src], dst)
        plan.execute([src], dst)
    for _ in range(3):
        dst.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(dst.cpu().numpy().view(np.uint16), want)


def test_plan_stats_count_algorithmic_bytes(B):
    full = W.full_configs()
    want = {
        "c2_fwd": (51380224, 51380224, 0),
        "c3": (402653184, 402653184, 0),
        "c4": (32112640, 36864000, 2375680 * 2),
        "c5": (51380224, 462422016, 0),
    }
    for name, (rd, wr, fl) in want.items():
        st = B.compose_chain(full[name]).plan(0).stats()
        assert (st["bytes_read"], st["bytes_written"], st["bytes_filled"]) == (rd, wr, fl), (name, st)


@pytest.mark.parametrize("name", ["c2_fwd", "c2_inv", "c3", "c3_merge", "c4", "c5"])
def test_full_size_configs_bit_exact(B, name):
    """The sizes and launch configuration the benchmark times."""
    chain = W.full_configs()[name]
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs, nt=min(os.cpu_count() or 1, 32))
    got, plan = run_gpu(B, chain, xs)
    assert np.array_equal(got, want.reshape(-1))
    del want, got
