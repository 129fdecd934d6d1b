"""Host algebra (amap_compose) on the CPU: the composed pieces, evaluated point
by point with a few lines of numpy, must reproduce the oracle's sequential
chain; plus the error paths and the C ABI's export list."""
import os
import re

import numpy as np
import pytest

from oracle import oracle
from paper_2002_12798_b200 import binding as B
from paper_2002_12798_b200 import workloads as W
from chain_gen import random_chain

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def eval_map(m, inputs):
    """Stage by stage: dst.flat[C_s i + b_s] = src.flat[C_l i + b_l] for every loop point of every piece."""
    flat = [x.reshape(-1) for x in inputs]
    pieces = m.pieces()
    result = None
    for first, n_pieces, dst_temp, numel in m.stages():
        if dst_temp < 0 and len(m.out_numels) > 1:  # the last stage of a map with several outputs
            result = [_eval_pieces([p for p in pieces[first : first + n_pieces] if p["output"] == k], n, flat, inputs[0].dtype)
                      for k, n in enumerate(m.out_numels)]
            continue
        out = _eval_pieces(pieces[first : first + n_pieces], numel, flat, inputs[0].dtype)
        if dst_temp >= 0:
            assert dst_temp == len(flat) - len(inputs), "temporaries are numbered in the order they are written"
            flat.append(out)
        else:
            result = out
    assert result is not None and m.stages()[-1][2] == -1
    return result


def _eval_pieces(pieces, numel, flat, dtype):
    if True:
        out = np.zeros(numel, dtype=dtype)
        cnt = np.zeros(numel, dtype=np.int32)
        for p in pieces:
            nl = len(p["bounds"])
            idx = np.indices(p["bounds"], dtype=np.int64).reshape(nl, -1) if nl else np.zeros((0, 1), dtype=np.int64)

            def aff(c, c0):
                v = np.full(idx.shape[1], c0, dtype=np.int64)
                for k, ck in enumerate(c):
                    v += ck * idx[k]
                return v

            dom = np.ones(idx.shape[1], bool)
            for c, o, e in p["domain"]:
                v = aff(c, o)
                dom &= (v >= 0) & (v < e)
            g = np.ones(idx.shape[1], bool)
            for c, o, e in p["guards"]:
                v = aff(c, o)
                g &= (v >= 0) & (v < e)
            d = aff(p["C_s"], p["b_s"])[dom]
            if p["input"] >= 0:
                s = aff(p["C_l"], p["b_l"])
                if p["quasi"]:  # b_l + sum_k stride_k * digit_k(f0 + F i), digits in the mixed radix, innermost last
                    f = aff(p["quasi"]["F"], p["quasi"]["f0"])
                    f = np.where(dom & g, f, 0)
                    for radix, stride in zip(reversed(p["quasi"]["radix"][1:]), reversed(p["quasi"]["stride"][1:])):
                        s += stride * (f % radix)
                        f = f // radix
                    assert ((f >= 0) & (f < p["quasi"]["radix"][0])).all()
                    s += p["quasi"]["stride"][0] * f
                s = s[dom]
                gg = g[dom]
                vals = np.where(gg, flat[p["input"]][np.where(gg, s, 0)], p["fill_bits"]).astype(out.dtype)
            else:
                vals = np.full(d.shape, p["fill_bits"], dtype=out.dtype)
            out[d] = vals
            np.add.at(cnt, d, 1)
        assert (cnt == 1).all(), "the pieces of a stage must write every element exactly once"
        return out


@pytest.mark.parametrize("name", sorted(W.reduced_configs()))
def test_composed_map_equals_sequential_chain(name):
    chain = W.reduced_configs()[name]
    xs = W.make_inputs(chain)
    m = B.compose_chain(chain)
    want = oracle.run_chain(chain, xs)
    assert m.out_numel == want.size and m.elem_size == chain.elem_size
    assert np.array_equal(eval_map(m, xs), want.reshape(-1))


def test_c1_composes_to_the_closed_form():
    (p,) = B.compose_chain(W.c1_small_chain()).pieces()
    # loops (a, j, k) < (64, 8, 6): load X.flat[2a + 1024j + 128k + 128], store Y.flat[48a + 6j + k]
    assert p["bounds"] == [64, 8, 6]
    assert p["C_l"] == [2, 1024, 128] and p["b_l"] == 128
    assert p["C_s"] == [48, 6, 1] and p["b_s"] == 0
    assert not p["guards"] and not p["domain"]


def test_full_size_maps_have_the_expected_shape():
    full = W.full_configs()
    (p,) = B.compose_chain(full["c2_fwd"]).pieces()
    assert (p["bounds"], p["C_l"], p["C_s"]) == ([32, 3136, 256], [802816, 1, 3136], [802816, 256, 1])
    (p,) = B.compose_chain(full["c2_inv"]).pieces()
    assert (p["bounds"], p["C_l"], p["C_s"]) == ([32, 256, 3136], [802816, 1, 256], [802816, 3136, 1])
    p0, p1 = B.compose_chain(full["c3"]).pieces()
    assert p0["bounds"] == p1["bounds"] == [16, 32, 1536, 128]
    assert p0["C_l"] == [8388608, 128, 4096, 1] and p0["C_s"] == [12582912, 393216, 128, 1]
    assert (p0["b_s"], p1["b_s"], p0["input"], p1["input"]) == (0, 196608, 0, 1)
    (p,) = B.compose_chain(full["c5"]).pieces()
    assert p["bounds"] == [64, 56, 56, 3, 3, 128]
    assert p["C_l"] == [401408, 7168, 128, 7168, 128, 1] and p["b_l"] == -7296
    assert p["C_s"] == [3612672, 64512, 1152, 384, 128, 1]
    assert len(p["guards"]) == 2 and not p["domain"]
    c4 = B.compose_chain(full["c4"]).pieces()
    copies = [p for p in c4 if p["input"] >= 0]
    assert sorted(p["bounds"][-1] for p in copies) == [32, 64, 96, 128]
    for p in copies:
        cq = p["bounds"][-1]
        assert p["bounds"] == [64, 28, 28, cq] and p["C_l"] == [784 * cq, 28, 1, 784] and p["C_s"] == [288000, 9600, 320, 1]
    filled = sum(int(np.prod(p["bounds"])) for p in c4 if p["input"] < 0)
    assert filled == 2375680


def test_random_tiny_chains():
    r = np.random.default_rng(12798)
    done = unsupported = 0
    for trial in range(300):
        chain = random_chain(r)
        xs = [x + np.uint32(1) for x in W.make_index_tagged_inputs(chain)]
        m = B.compose_chain(chain)  # every valid chain composes; what cannot be eliminated stays as a temporary
        unsupported += len(m.stages()) > 1
        want = oracle.run_chain(chain, xs)
        assert np.array_equal(eval_map(m, xs), want.reshape(-1)), (trial, chain.ops)
        done += 1
    assert done == 300 and unsupported < 100, (done, unsupported)


def test_pad_written_as_explicit_fill_statements():
    """The other encoding of padding: border boxes of constant stores plus an interior copy."""
    b = B.Builder(2)
    x = b.input([4, 5])
    t = b.tensor([6, 8])  # pad 1 on axis 0, (1, 2) on axis 1
    eye = [[1, 0], [0, 1]]
    b.stmt([1, 8], None, (t, eye, [0, 0]), fill_bits=7)
    b.stmt([1, 8], None, (t, eye, [5, 0]), fill_bits=7)
    b.stmt([4, 1], None, (t, eye, [1, 0]), fill_bits=7)
    b.stmt([4, 2], None, (t, eye, [1, 6]), fill_bits=7)
    b.stmt([4, 5], (x, eye, [0, 0]), (t, eye, [1, 1]))
    y = b.transpose(t, [1, 0])
    m = b.compose(y)
    xin = np.arange(1, 21, dtype=np.uint16).reshape(4, 5)
    want = np.pad(xin, [(1, 1), (1, 2)], constant_values=7).T
    assert np.array_equal(eval_map(m, [xin]).reshape(8, 6), want)


def test_window_over_a_transposed_input_stays_one_guarded_piece():
    b = B.Builder(2)
    x = b.input([2, 3, 6, 5])  # NCHW
    nhwc = b.transpose(x, [0, 2, 3, 1])
    y = b.window(nhwc, 3, 3, 1, 1)
    m = b.compose(y)
    ps = m.pieces()
    assert len(ps) == 1 and len(ps[0]["guards"]) == 2
    xin = np.random.default_rng(3).integers(1, 60000, size=(2, 3, 6, 5)).astype(np.uint16)
    want = oracle.window(oracle.transpose(xin, [0, 2, 3, 1]), 3, 3, 1, 1)
    assert np.array_equal(eval_map(m, [xin]), want.reshape(-1))


def test_a_5x5_window_is_one_guarded_piece():
    """A 5x5 window with stride 1 and padding 2 composes to one piece with two guards (as the 3x3 one does)."""
    b = B.Builder(2)
    x = b.input([2, 9, 8, 4])
    m = b.compose(b.window(x, 5, 5, 1, 2))
    ps = m.pieces()
    assert len(ps) == 1 and len(ps[0]["guards"]) == 2
    xin = np.random.default_rng(4).integers(1, 60000, size=(2, 9, 8, 4)).astype(np.uint16)
    assert np.array_equal(eval_map(m, [xin]), oracle.window(xin, 5, 5, 1, 2).reshape(-1))


def test_an_intermediate_with_two_readers_is_eliminated_for_both():
    """A small DAG: one transposed tensor feeds a slice and a pad, whose results are joined again.  The shared
    intermediate has two readers; each is rewritten against it (Section 2.1, equation (2), per reader)."""
    b = B.Builder(2)
    x = b.input([6, 10])
    t = b.transpose(x, [1, 0])                        # [10, 6], read twice below
    left = b.slice(t, [0, 0], [10, 4], [1, 2])        # [10, 2]
    right = b.pad(t, [0, 0], [0, 3])                  # [10, 9]
    m = b.compose(b.concat([left, right, left], 1))   # [10, 13]
    assert len(m.stages()) == 1
    xin = np.random.default_rng(11).integers(1, 60000, size=(6, 10)).astype(np.uint16)
    tt = xin.T
    want = np.concatenate([tt[:, 0:4:2], np.pad(tt, [(0, 0), (0, 3)]), tt[:, 0:4:2]], 1)
    assert np.array_equal(eval_map(m, [xin]), want.reshape(-1))
    ot = oracle.transpose(xin, [1, 0])
    ol = oracle.slice_(ot, [0, 0], [10, 4], [1, 2])
    assert np.array_equal(oracle.concat([ol, oracle.pad(ot, [0, 0], [0, 3]), ol], 1), want)


def test_tile_is_a_broadcast_load():
    b = B.Builder(4)
    x = b.input([2, 3])
    y = b.tile(x, [2, 3])
    m = b.compose(b.transpose(y, [1, 0]))
    xin = np.arange(6, dtype=np.uint32).reshape(2, 3) + 1
    assert np.array_equal(eval_map(m, [xin]).reshape(9, 4), np.tile(xin, (2, 3)).T)


# ---------------------------------------------------------------------------
# error paths (all on the host)
# ---------------------------------------------------------------------------
def _code(fn):
    with pytest.raises(B.AmapError) as e:
        fn()
    return e.value.code


def test_error_codes():
    eye = [[1, 0], [0, 1]]

    def non_injective():
        b = B.Builder(4)
        x = b.input([4, 4])
        t = b.tensor([4])
        b.stmt([4, 4], (x, eye, [0, 0]), (t, [[1, 0]], [0]))  # the second loop never moves the store
        b.compose(t)

    assert _code(non_injective) == -2

    def interleaved_collision():
        b = B.Builder(4)
        x = b.input([4, 4])
        t = b.tensor([16])
        b.stmt([4, 4], (x, eye, [0, 0]), (t, [[2, 3]], [0]))  # 2a + 3b collides (a,b) = (3,0) and (0,2)
        b.compose(t)

    assert _code(interleaved_collision) == -2

    def load_escapes():
        b = B.Builder(4)
        x = b.input([4, 4])
        t = b.tensor([4, 4])
        b.stmt([4, 4], (x, eye, [1, 0]), (t, eye, [0, 0]))
        b.compose(t)

    assert _code(load_escapes) == -3

    def store_escapes():
        b = B.Builder(4)
        x = b.input([4, 4])
        t = b.tensor([4, 4])
        b.stmt([4, 4], (x, eye, [0, 0]), (t, eye, [0, 1]))
        b.compose(t)

    assert _code(store_escapes) == -3

    def output_partly_written():
        b = B.Builder(4)
        x = b.input([4, 4])
        t = b.tensor([4, 5])
        b.stmt([4, 4], (x, eye, [0, 0]), (t, eye, [0, 0]))
        b.compose(t)

    assert _code(output_partly_written) == -4

    def reads_unwritten_intermediate():
        b = B.Builder(4)
        x = b.input([4, 4])
        t = b.tensor([4, 5])
        b.stmt([4, 4], (x, eye, [0, 0]), (t, eye, [0, 0]))
        b.compose(b.transpose(t, [1, 0]))

    assert _code(reads_unwritten_intermediate) == -4

    def overlap():
        b = B.Builder(4)
        x = b.input([4, 4])
        t = b.tensor([4, 6])
        b.stmt([4, 4], (x, eye, [0, 0]), (t, eye, [0, 0]))
        b.stmt([4, 4], (x, eye, [0, 0]), (t, eye, [0, 2]))
        b.compose(t)

    assert _code(overlap) == -5

    assert _code(lambda: B.Builder(3)) == -1
    assert _code(lambda: B.Builder(4).reshape(0, [2])) == -1  # no such tensor


def test_reshape_whose_factors_do_not_line_up():
    """[4,6] -> transpose -> [6,4] -> reshape [8,3] -> transpose -> [3,8]: the reshape has no common refinement
    with the loops around it.  The library must still return the right answer, with a temporary if need be."""
    chain = W.Chain(
        name="awkward", dtype="fp32", inputs=[[4, 6]],
        ops=[
            {"kind": "transpose", "src": 0, "perm": [1, 0]},
            {"kind": "reshape", "src": 1, "shape": [8, 3]},
            {"kind": "transpose", "src": 2, "perm": [1, 0]},
        ],
        values="raw",
    )
    xs = W.make_index_tagged_inputs(chain)
    m = B.compose_chain(chain)
    assert np.array_equal(eval_map(m, xs), oracle.run_chain(chain, xs).reshape(-1))
    # two such reshapes in a row shatter the loops: the library keeps a temporary rather than dozens of pieces
    chain.inputs = [[40, 24]]
    chain.ops = [
        {"kind": "transpose", "src": 0, "perm": [1, 0]},
        {"kind": "reshape", "src": 1, "shape": [64, 15]},
        {"kind": "transpose", "src": 2, "perm": [1, 0]},
        {"kind": "reshape", "src": 3, "shape": [24, 40]},
        {"kind": "transpose", "src": 4, "perm": [1, 0]},
    ]
    xs = W.make_index_tagged_inputs(chain)
    m = B.compose_chain(chain)
    assert len(m.stages()) >= 2
    assert np.array_equal(eval_map(m, xs), oracle.run_chain(chain, xs).reshape(-1))
    # a lone reshape of that kind needs no temporary: it is one flat loop
    b = B.Builder(4)
    x = b.input([2, 3])
    m = b.compose(b.reshape(x, [3, 2]))
    assert len(m.stages()) == 1 and len(m.pieces()) == 1


def test_no_fuse_keeps_every_intermediate():
    """The unfused chain (one stage per operator) gives the same bytes as the composed map."""
    for name in ("c1", "c3_odd", "c4_odd", "c5_odd"):
        chain = W.reduced_configs()[name]
        xs = W.make_inputs(chain)
        fused, unfused = B.compose_chain(chain), B.compose_chain(chain, B.COMPOSE_NO_FUSE)
        assert len(fused.stages()) == 1
        n_ops = len(chain.ops)
        assert len(unfused.stages()) == n_ops, name
        want = oracle.run_chain(chain, xs).reshape(-1)
        assert np.array_equal(eval_map(fused, xs), want) and np.array_equal(eval_map(unfused, xs), want)


def test_interleaved_stores_are_told_apart_from_overlap():
    b = B.Builder(2)
    x0, x1 = b.input([8]), b.input([8])
    t = b.tensor([16])
    b.stmt([8], (x0, [[1]], [0]), (t, [[2]], [0]))
    b.stmt([8], (x1, [[1]], [0]), (t, [[2]], [1]))
    m = b.compose(b.reshape(t, [4, 4]))
    a, c = np.arange(8, dtype=np.uint16) + 100, np.arange(8, dtype=np.uint16) + 200
    want = np.empty(16, np.uint16)
    want[0::2], want[1::2] = a, c
    assert np.array_equal(eval_map(m, [a, c]), want)


def test_huge_pieces_are_cut_below_2_31_points():
    """An 18 GB byte tensor (shapes only, nothing is allocated): the planner's 32-bit item index must still cover it."""
    b = B.Builder(1)
    x = b.input([3, 1 << 16, 3 << 15])
    m = b.compose(b.transpose(b.slice(x, [0, 0, 1], [3, 1 << 16, 3 << 15], [1, 1, 2]), [1, 0, 2]))
    ps = m.pieces()
    assert len(ps) > 1 and all(int(np.prod(p["bounds"], dtype=np.int64)) < 2**31 for p in ps)
    assert sum(int(np.prod(p["bounds"], dtype=np.int64)) for p in ps) == m.out_numel
    st = m.plan(device=-1).stats()  # the dry plan walks sampled addresses of every descriptor
    assert st["bytes_written"] == m.out_numel


def test_empty_and_scalar_shapes():
    b = B.Builder(2)
    x = b.input([1, 1])
    m = b.compose(b.transpose(x, [1, 0]))
    assert np.array_equal(eval_map(m, [np.array([[9]], np.uint16)]), [9])
    b = B.Builder(2)
    x = b.input([0, 3])
    m = b.compose(b.transpose(x, [1, 0]))
    assert m.out_numel == 0 and m.pieces() == []


# ---------------------------------------------------------------------------
# the C ABI
# ---------------------------------------------------------------------------
def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "amap.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(amap_[a-z_]+)\s*\(", header))
    assert declared and declared == set(B.EXPORTS), declared ^ set(B.EXPORTS)
    import ctypes

    lib = ctypes.CDLL(B.LIBRARY_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert lib.amap_strerror  # loads without a GPU


def test_strerror_is_distinct_per_code():
    import ctypes

    lib = ctypes.CDLL(B.LIBRARY_PATH)
    lib.amap_strerror.restype = ctypes.c_char_p
    msgs = {lib.amap_strerror(c) for c in range(0, -11, -1)}
    assert len(msgs) == 11


# ---------------------------------------------------------------------------
# several outputs from one compose, and operators that are not layout operators
# ---------------------------------------------------------------------------
def _qkv_chain(Bt=2, S=12, heads=3, D=8):
    hd = heads * D
    ops = []
    for part in range(3):
        base = 1 + len(ops)
        ops.append({"kind": "split", "src": 0, "axis": 2, "sizes": [hd, hd, hd], "part": part})
        ops.append({"kind": "reshape", "src": base, "shape": [Bt, S, heads, D]})
        ops.append({"kind": "transpose", "src": base + 1, "perm": [0, 2, 1, 3]})
    return W.Chain(name="qkv", dtype="bf16", inputs=[[Bt, S, 3 * hd]], ops=ops, values="normal"), [3, 6, 9]


def test_split_parts_compose_into_one_map_with_three_outputs():
    chain, outs = _qkv_chain()
    xs = W.make_inputs(chain)
    tensors = oracle.run_chain(chain, xs, keep_intermediates=True)
    m = B.compose_chain(chain, outputs=outs)
    assert len(m.out_numels) == 3 and len(m.stages()) == 1
    got = eval_map(m, xs)
    for k, t in enumerate(outs):
        assert np.array_equal(got[k], tensors[t].reshape(-1)), k
    st = m.plan(device=-1).stats()
    assert st["n_launches"] == 1 and st["n_stages"] == 1  # one launch writes q, k and v
    assert st["bytes_written"] == sum(m.out_numels) * 2 and st["bytes_read"] == xs[0].nbytes


def test_a_tensor_can_be_an_output_and_be_read_again():
    chain = W.Chain(
        name="both", dtype="fp32", inputs=[[6, 10]],
        ops=[
            {"kind": "transpose", "src": 0, "perm": [1, 0]},                 # 1: [10, 6], an output
            {"kind": "pad", "src": 1, "lo": [1, 0], "hi": [0, 2]},           # 2: [11, 8], an output too
            {"kind": "slice", "src": 1, "start": [2, 1], "stop": [9, 6], "step": [3, 2]},  # 3: a third
        ],
        values="raw",
    )
    xs = W.make_index_tagged_inputs(chain)
    tensors = oracle.run_chain(chain, xs, keep_intermediates=True)
    m = B.compose_chain(chain, outputs=[2, 1, 3])  # in the order asked for
    got = eval_map(m, xs)
    for k, t in enumerate([2, 1, 3]):
        assert np.array_equal(got[k], tensors[t].reshape(-1))
    assert [p["input"] for p in m.pieces() if p["input"] >= 0] == [0] * sum(p["input"] >= 0 for p in m.pieces())


def test_outputs_are_validated():
    b = B.Builder(4)
    x = b.input([4, 6])
    y = b.transpose(x, [1, 0])
    z = b.reshape(y, [3, 8])
    for outs in ([y, y], [x, y], [], [99], [y] * 9):
        with pytest.raises(B.AmapError) as e:
            b.compose_multi(outs)
        assert e.value.code == -1
    assert len(b.compose_multi([z, y]).out_numels) == 2


def test_composition_stops_at_an_operator_that_is_not_a_layout_operator():
    """x -> transpose -> [compute operator] -> pad -> transpose.  The statements before the operator compose into its
    input (asked for as an output), the statements behind it into reads of its result (bound like an input)."""
    b = B.Builder(2)
    x = b.input([8, 20])
    t = b.transpose(b.reshape(x, [8, 4, 5]), [2, 0, 1])        # [5, 8, 4]: what the operator consumes
    o = b.opaque([t], [5, 8, 4])                                # its result
    z = b.transpose(b.pad(o, [0, 1, 0], [0, 0, 2]), [1, 0, 2])  # [9, 5, 6]
    first = b.compose_multi([t])
    second = b.compose(z)
    xv = np.arange(160, dtype=np.uint16).reshape(8, 20)
    tv = eval_map(first, [xv])
    assert np.array_equal(tv, xv.reshape(8, 4, 5).transpose(2, 0, 1).reshape(-1))
    ov = (tv.astype(np.uint32) * 3 + 7).astype(np.uint16)      # stands in for the compute operator
    zv = eval_map(second, [xv, ov])
    want = np.pad(ov.reshape(5, 8, 4), ((0, 0), (1, 0), (0, 2))).transpose(1, 0, 2)
    assert np.array_equal(zv, want.reshape(-1))
    assert all(p["input"] in (1, -1) for p in second.pieces())  # nothing behind the operator reads x
    # one compose cannot reach through the operator: a map that wants z never reads the transposed tensor
    assert second.in_numel == [160, 160]


# ---------------------------------------------------------------------------
# the map flattened for a consumer kernel (include/amap_device.h)
# ---------------------------------------------------------------------------
def eval_view(v, inputs):
    """What amap_view_locate computes, for every output index at once: decode the index into a piece's loop indices
    digit by digit, check the constraints, follow the source strides."""
    flat = [x.reshape(-1) for x in inputs]
    o = np.arange(v.out_numel, dtype=np.int64)
    out = np.zeros(v.out_numel, dtype=inputs[0].dtype)
    hit = np.zeros(v.out_numel, dtype=np.int32)
    for q in range(v.n_pieces):
        pc = v.piece[q]
        rem = o - pc.b_s
        ok = rem >= 0
        idx = []
        for k in range(pc.n_loops):
            i = np.where(ok, rem // pc.dst_stride[k], 0)
            ok &= i < pc.ext[k]
            idx.append(i)
            rem = rem - i * pc.dst_stride[k]
        ok &= rem == 0
        load = np.full(v.out_numel, pc.input >= 0)
        for c in range(pc.n_guards + pc.n_domain):
            e = np.full(v.out_numel, pc.cons[c].offset, dtype=np.int64)
            for k in range(pc.n_loops):
                e += pc.cons[c].coef[k] * idx[k]
            good = (e >= 0) & (e < pc.cons[c].extent)
            if c < pc.n_guards:
                load &= good
            else:
                ok &= good
        s = np.full(v.out_numel, pc.b_l, dtype=np.int64)
        for k in range(pc.n_loops):
            s += pc.src_stride[k] * idx[k]
        take = ok & load
        if pc.input >= 0:
            out[take] = flat[pc.input][s[take]]
        out[ok & ~load] = pc.fill_bits
        hit += ok
    assert (hit == 1).all(), "every output index must decode into exactly one piece"
    return out


@pytest.mark.parametrize("name", ["c1", "c2_fwd", "c2_inv_odd_f32", "c3", "c3_odd", "c4", "c4_odd", "c5", "c5_odd", "c5_dil2", "c5_crs"])
def test_device_view_reproduces_the_chain(name):
    chain = W.reduced_configs()[name]
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs)
    m = B.compose_chain(chain)
    v = m.device_view()
    assert v.out_numel == m.out_numel and v.elem_size == chain.elem_size and v.n_inputs == len(xs)
    assert np.array_equal(eval_view(v, xs), want.reshape(-1))


@pytest.mark.parametrize("name,cols,whole_runs", [
    ("c5", 9 * 128, True), ("c5", 3 * 128, True), ("c5", 128, True), ("c5_odd", 9 * 24, True), ("c5_dil2", None, True),
    ("c3", 128, True), ("c3", 2 * 128, True), ("c3_odd", 24, True), ("c3_odd", 17 * 24, True),
    ("c5_crs", None, False),  # columns ordered (c, r, s): the innermost loop strides the source
    ("c2_inv", 11, False), ("c1", 16, False),  # strided sources
    ("c4", 320, None), ("c4_odd", 88, None), ("c2_inv", 13 * 11, None), ("c1", 48, None),
])
def test_row_tables_reproduce_the_chain(name, cols, whole_runs):
    """The consumer's row walk (outer loops decoded once per row, the runs inside a row from a table) on the host:
    rows of one run, of several runs with guards (window gathers), rows that cut a loop in two, rows that span a
    whole inner nest.  `whole_runs`: whether the rows are known to be whole runs (None: either answer is fine, the
    result must be right if there is one)."""
    chain = W.reduced_configs()[name]
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs)
    m = B.compose_chain(chain)
    cols = cols or want.shape[-1]
    try:
        got = m.rows_gather_host(xs, cols)
    except B.AmapError as e:
        assert e.code == -9 and not whole_runs, e  # the functor's job
        return
    assert whole_runs is not False
    assert np.array_equal(got.view(np.uint8), np.ascontiguousarray(want).reshape(-1).view(np.uint8))


def test_row_tables_of_a_plain_copy_split_its_one_loop():
    b = B.Builder(2)
    m = b.compose(b.reshape(b.input([6, 40]), [240]))
    x = np.arange(240, dtype=np.uint16)
    for cols in (240, 40, 8, 1):
        assert np.array_equal(m.rows_gather_host([x], cols), x)
    with pytest.raises(B.AmapError):
        m.rows_gather_host([x], 7)  # does not divide the result


def test_device_view_refuses_what_it_cannot_hold():
    b = B.Builder(2)
    ids = [b.input([4, 8]) for _ in range(5)]
    m = b.compose(b.concat([b.pad(t, [1, 1], [1, 1]) for t in ids], 0))  # far more than 8 pieces
    with pytest.raises(B.AmapError) as e:
        m.device_view()
    assert e.value.code == -11
    chain, outs = _qkv_chain()
    with pytest.raises(B.AmapError) as e:
        B.compose_chain(chain, outputs=outs).device_view()  # several outputs
    assert e.value.code == -9


# ---------------------------------------------------------------------------
# quasi-affine pieces: reshapes whose factors do not line up with the loops around them
# ---------------------------------------------------------------------------
def _run_preserving_chain(a=100, b=81, c=90, d=90, inner=8, dtype="bf16"):
    """[a, b, inner] -> transpose(1,0,2) -> reshape [c, d, inner] (a*b == c*d, the factors do not line up) ->
    transpose(1,0,2): rows of `inner` elements stay contiguous on both sides."""
    assert a * b == c * d
    return W.Chain(
        name="quasi_runs", dtype=dtype, inputs=[[a, b, inner]],
        ops=[
            {"kind": "transpose", "src": 0, "perm": [1, 0, 2]},
            {"kind": "reshape", "src": 1, "shape": [c, d, inner]},
            {"kind": "transpose", "src": 2, "perm": [1, 0, 2]},
        ],
        values="normal",
    )


def _scattered_chain(m=128, n=90, r=160):
    """[m, n] -> transpose -> reshape [r, m*n/r] -> transpose: no contiguous run survives."""
    return W.Chain(
        name="quasi_scattered", dtype="bf16", inputs=[[m, n]],
        ops=[
            {"kind": "transpose", "src": 0, "perm": [1, 0]},
            {"kind": "reshape", "src": 1, "shape": [r, m * n // r]},
            {"kind": "transpose", "src": 2, "perm": [1, 0]},
        ],
        values="normal",
    )


def test_runs_that_survive_a_misaligned_reshape_compose_into_one_quasi_affine_piece():
    chain = _run_preserving_chain()
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs)
    m = B.compose_chain(chain)
    assert len(m.stages()) == 1  # no temporary
    quasi = [p for p in m.pieces() if p["quasi"]]
    assert len(quasi) == 1 and quasi[0]["quasi"]["radix"][-1] == 8 and quasi[0]["quasi"]["stride"][-1] == 1
    assert np.array_equal(eval_map(m, xs), want.reshape(-1))
    st = m.plan(device=-1).stats()
    assert st["n_stages"] == 1 and st["kernels"]["copy"] == 1  # 16-byte units: one division chain per unit
    # switched off, the pair keeps its temporary
    m2 = B.compose_chain(chain, B.COMPOSE_NO_QUASI_AFFINE)
    assert len(m2.stages()) == 2 and not any(p["quasi"] for p in m2.pieces())
    assert np.array_equal(eval_map(m2, xs), want.reshape(-1))


def test_scattered_quasi_affine_pairs_keep_their_temporary_unless_forced():
    chain = _scattered_chain()
    xs = W.make_inputs(chain)
    want = oracle.run_chain(chain, xs)
    m = B.compose_chain(chain)
    assert len(m.stages()) == 2 and not any(p["quasi"] for p in m.pieces())
    forced = B.compose_chain(chain, B.COMPOSE_QUASI_AFFINE)
    assert len(forced.stages()) == 1 and any(p["quasi"] for p in forced.pieces())
    assert np.array_equal(eval_map(forced, xs), want.reshape(-1))
    assert forced.plan(device=-1).stats()["kernels"]["gather"] == 1


def test_readers_of_a_quasi_affine_tensor_and_guards_compose_on():
    """pad and slice behind the misaligned reshape: the reader's guards stay affine in its own loops, and a reader
    that lines up with the quasi-affine writer inherits its digits."""
    chain = _run_preserving_chain(dtype="fp32")
    chain.ops += [
        {"kind": "pad", "src": 3, "lo": [1, 0, 0], "hi": [0, 2, 0]},
        {"kind": "slice", "src": 4, "start": [0, 1, 0], "stop": [91, 90, 8], "step": [3, 2, 1]},
    ]
    chain.values = "raw"
    xs = W.make_index_tagged_inputs(chain)
    xs = [x + np.uint32(1) for x in xs]
    want = oracle.run_chain(chain, xs)
    for flags in (0, B.COMPOSE_QUASI_AFFINE):
        m = B.compose_chain(chain, flags)
        assert np.array_equal(eval_map(m, xs), want.reshape(-1))
    assert len(B.compose_chain(chain).stages()) == 1


def test_random_chains_with_quasi_affine_composition_forced():
    r = np.random.default_rng(1279800)
    quasi = 0
    for trial in range(300):
        chain = random_chain(r)
        xs = [x + np.uint32(1) for x in W.make_index_tagged_inputs(chain)]
        try:
            m = B.compose_chain(chain, B.COMPOSE_QUASI_AFFINE)
        except B.AmapError as e:
            assert e.code == -9
            continue
        quasi += any(p["quasi"] for p in m.pieces())
        want = oracle.run_chain(chain, xs)
        assert np.array_equal(eval_map(m, xs), want.reshape(-1)), (trial, chain.ops)
        m.plan(device=-1)  # the planner's host replay of every address
    assert quasi >= 10
