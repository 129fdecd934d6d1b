"""Pins for the CPU oracle: every check here compares it with something that is
not the oracle -- hand-derived closed forms, invariants of permutations,
numpy / torch library routines on special cases, and brute force in Python."""
import itertools
import os

import numpy as np
import pytest

from oracle import oracle
from paper_2002_12798_b200 import workloads as W
from chain_gen import random_chain

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(7)


def rand_u(shape, dtype=np.uint16):
    info = np.iinfo(dtype)
    return rng.integers(1, info.max, size=shape, dtype=dtype)  # never 0: zeros mean padding


# ---------------------------------------------------------------------------
# configuration 1: hand-derived closed form (tests/golden/c1_closed_form.txt)
# ---------------------------------------------------------------------------
def test_c1_golden_values():
    chain = W.c1_small_chain()
    out = oracle.run_chain(chain, W.make_index_tagged_inputs(chain))
    assert out.shape == (64, 48)
    n = 0
    for line in open(os.path.join(GOLDEN, "c1_closed_form.txt")):
        if line.startswith("#") or not line.strip():
            continue
        r, c, v = (int(t) for t in line.split())
        assert int(out[r, c]) == v, (r, c)
        n += 1
    assert n == 12


def test_c1_closed_form_everywhere():
    chain = W.c1_small_chain()
    out = oracle.run_chain(chain, W.make_index_tagged_inputs(chain))
    a, j, k = np.meshgrid(np.arange(64), np.arange(8), np.arange(6), indexing="ij")
    want = np.zeros((64, 48), dtype=np.int64)
    want[a, 6 * j + k] = 1024 * j + 128 * k + 128 + 2 * a
    assert np.array_equal(out.astype(np.int64), want)


def test_c1_seeded_values_follow_the_index_map():
    chain = W.c1_small_chain()
    (x,) = W.make_inputs(chain)
    src = oracle.run_chain(chain, W.make_index_tagged_inputs(chain)).astype(np.int64)
    out = oracle.run_chain(chain, [x])
    assert np.array_equal(out, x.reshape(-1)[src])
    # the recipe: integers below 2**20 stored as fp32
    f = x.view(np.float32)
    assert f.min() >= 0 and f.max() < 2**20 and np.array_equal(f, np.round(f))


# ---------------------------------------------------------------------------
# reshape, transpose
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("es_dtype", [np.uint8, np.uint16, np.uint32, np.uint64])
def test_reshape_is_flat_identity(es_dtype):
    x = rand_u((6, 10, 7), es_dtype)
    y = oracle.reshape(x, [3, 4, 35])
    assert y.shape == (3, 4, 35)
    assert y.tobytes() == x.tobytes()
    with pytest.raises(ValueError):
        oracle.reshape(x, [3, 4, 36])


@pytest.mark.parametrize("perm", list(itertools.permutations(range(4)))[::3])
def test_transpose_matches_numpy_and_is_a_bijection(perm):
    x = np.arange(3 * 4 * 5 * 6, dtype=np.uint32).reshape(3, 4, 5, 6)
    y = oracle.transpose(x, perm)
    assert y.shape == tuple(x.shape[p] for p in perm)
    assert np.array_equal(y, np.transpose(x, perm))
    assert np.array_equal(np.sort(y.reshape(-1)), x.reshape(-1))  # every element exactly once
    inv = np.argsort(perm)
    assert np.array_equal(oracle.transpose(y, list(inv)), x)  # perm then its inverse = identity


def test_transpose_twice_is_identity_and_keeps_bits():
    # NaN payloads and negative zero are plain bit patterns here
    x = np.array([[0x7FC00001, 0x80000000, 0xFFFFFFFF], [1, 2, 3]], dtype=np.uint32)
    y = oracle.transpose(oracle.transpose(x, [1, 0]), [1, 0])
    assert y.tobytes() == x.tobytes()


def test_nchw_nhwc_round_trip():
    fwd, inv = W.c2_nchw_to_nhwc(N=2, C=5, H=4, W=3), W.c2_nhwc_to_nchw(N=2, C=5, H=4, W=3)
    (x,) = W.make_inputs(fwd)
    y = oracle.run_chain(fwd, [x])
    assert y.shape == (2, 4, 3, 5)
    n, c, h, w = 1, 3, 2, 1
    assert y[n, h, w, c] == x[n, c, h, w]
    assert np.array_equal(y, np.transpose(x, (0, 2, 3, 1)))
    assert np.array_equal(oracle.run_chain(inv, [y]), x)


def test_transpose_rejects_a_non_permutation():
    with pytest.raises(ValueError):
        oracle.transpose(np.zeros((2, 3), np.uint16), [0, 0])


# ---------------------------------------------------------------------------
# slice, pad, concat
# ---------------------------------------------------------------------------
def test_slice_matches_numpy():
    x = rand_u((9, 8, 7))
    y = oracle.slice_(x, [1, 0, 2], [9, 8, 7], [3, 1, 2])
    assert np.array_equal(y, x[1:9:3, 0:8:1, 2:7:2])
    assert y.shape == (3, 8, 3)


def test_pad_then_slice_is_identity_and_border_is_zero():
    x = rand_u((3, 4, 5))
    lo, hi = [1, 0, 2], [2, 1, 0]
    p = oracle.pad(x, lo, hi)
    assert p.shape == (6, 5, 7)
    assert np.array_equal(p, np.pad(x, list(zip(lo, hi))))
    back = oracle.slice_(p, lo, [l + s for l, s in zip(lo, x.shape)], [1, 1, 1])
    assert np.array_equal(back, x)
    assert int((p == 0).sum()) == p.size - x.size


def test_concat_pieces_come_back_by_slicing():
    xs = [rand_u((2, n, 3)) for n in (4, 1, 5)]
    y = oracle.concat(xs, 1)
    assert np.array_equal(y, np.concatenate(xs, 1))
    off = 0
    for x in xs:
        piece = oracle.slice_(y, [0, off, 0], [2, off + x.shape[1], 3], [1, 1, 1])
        assert np.array_equal(piece, x)
        off += x.shape[1]
    with pytest.raises(ValueError):
        oracle.concat([xs[0], rand_u((3, 4, 3))], 1)


def test_c3_closed_form():
    B, S, heads, D, keep = 2, 33, 5, 24, 17
    chain = W.c3_head_split(B=B, S=S, heads=heads, D=D, keep=keep)
    xs = W.make_inputs(chain)
    y = oracle.run_chain(chain, xs)
    assert y.shape == (B, heads, 2 * keep, D)
    b, h, s, d = np.meshgrid(np.arange(B), np.arange(heads), np.arange(2 * keep), np.arange(D), indexing="ij")
    stacked = np.stack(xs)  # [2, B, S, heads*D]
    want = stacked[s // keep, b, s % keep, D * h + d]
    assert np.array_equal(y, want)
    # the opposite direction undoes the split of one tensor
    merge = W.c3_head_merge(B=B, S=2 * keep, heads=heads, D=D)
    z = oracle.run_chain(merge, [y])
    assert np.array_equal(z[:, :keep], xs[0][:, :keep])
    assert np.array_equal(z[:, keep:], xs[1][:, :keep])


def test_c4_matches_numpy_and_counts_its_zero_border():
    chain = W.c4_inception_concat()  # full size: 64 x (64|96|128|32) x 28 x 28
    xs = [rand_u(s) for s in chain.inputs]
    y = oracle.run_chain(chain, xs, nt=os.cpu_count() or 1)
    assert y.shape == (64, 30, 30, 320)
    assert int((y == 0).sum()) == 64 * 320 * (30 * 30 - 28 * 28) == 2375680
    want = np.concatenate([np.pad(x, [(0, 0), (0, 0), (1, 1), (1, 1)]) for x in xs], 1).transpose(0, 2, 3, 1)
    assert np.array_equal(y, want)
    # spot formula: Y[n, h+1, w+1, o_q + c] = X_q[n, c, h, w]
    assert y[5, 1 + 27, 1 + 0, 64 + 96 + 127] == xs[2][5, 127, 27, 0]


# ---------------------------------------------------------------------------
# window gather (im2col)
# ---------------------------------------------------------------------------
def test_window_1x1_is_a_reshape():
    x = rand_u((2, 5, 4, 3))
    y = oracle.window(x, 1, 1, 1, 0)
    assert y.shape == (40, 3) and y.tobytes() == x.tobytes()


def test_window_centre_tap_sum_identity_and_zero_count():
    N, H, Wd, C = 2, 9, 8, 6
    x = rng.integers(1, 1000, size=(N, H, Wd, C)).astype(np.uint32)
    y = oracle.window(x, 3, 3, 1, 1)
    assert y.shape == (N * H * Wd, 9 * C)
    # centre tap (r, s) = (1, 1) reproduces the input
    assert np.array_equal(y[:, 4 * C : 5 * C].reshape(x.shape), x)
    # each input element is used m(h) * m(w) times: 2 on an edge row/column, else 3
    mh = np.where((np.arange(H) == 0) | (np.arange(H) == H - 1), 2, 3)
    mw = np.where((np.arange(Wd) == 0) | (np.arange(Wd) == Wd - 1), 2, 3)
    want_sum = int((x.astype(np.int64) * mh[None, :, None, None] * mw[None, None, :, None]).sum())
    assert int(y.astype(np.int64).sum()) == want_sum
    # zero entries come only from the padding
    assert int((y == 0).sum()) == (9 * H * Wd - (3 * H - 2) * (3 * Wd - 2)) * N * C


def test_window_zero_count_formula_of_the_full_configuration():
    # (9*56^2 - (3*56-2)^2) * 64 * 128 zero entries at full size; checked here on the same geometry, 1 image, 2 channels
    x = rand_u((1, 56, 56, 2))
    y = oracle.window(x, 3, 3, 1, 1)
    assert int((y == 0).sum()) == (9 * 56 * 56 - (3 * 56 - 2) ** 2) * 2
    assert (9 * 56 * 56 - (3 * 56 - 2) ** 2) * 64 * 128 == 5472256


@pytest.mark.parametrize("k,stride,padding", [(3, 1, 1), (3, 2, 1), (2, 1, 0), (5, 2, 2)])
def test_window_matches_torch_unfold(k, stride, padding):
    torch = pytest.importorskip("torch")
    N, H, Wd, C = 2, 9, 7, 4
    x = rng.integers(1, 2000, size=(N, H, Wd, C)).astype(np.uint32)
    y = oracle.window(x, k, k, stride, padding)
    xt = torch.from_numpy(x.astype(np.float32)).permute(0, 3, 1, 2)  # NCHW
    u = torch.nn.functional.unfold(xt, k, padding=padding, stride=stride)  # [N, C*k*k, L], rows ordered (c, r, s)
    L = u.shape[-1]
    u = u.reshape(N, C, k, k, L).permute(0, 4, 2, 3, 1).reshape(N * L, k * k * C)  # -> (r, s, c) columns
    assert np.array_equal(y.astype(np.float32), u.numpy())


@pytest.mark.parametrize("k,stride,padding,dilation", [(3, 1, 2, 2), (3, 2, 2, 2), (2, 1, 1, 3), (3, 1, 1, 1), (5, 1, 4, 2)])
@pytest.mark.parametrize("order", ["rsc", "crs"])
def test_dilated_window_and_column_orders_match_torch_unfold(k, stride, padding, dilation, order):
    """torch's unfold has the dilation argument and produces the (c, r, s) column order natively."""
    torch = pytest.importorskip("torch")
    N, H, Wd, C = 2, 11, 9, 5
    x = rng.integers(1, 2000, size=(N, H, Wd, C)).astype(np.uint32)
    y = oracle.window(x, k, k, stride, padding, dilation=dilation, order=order)
    xt = torch.from_numpy(x.astype(np.float32)).permute(0, 3, 1, 2)  # NCHW
    u = torch.nn.functional.unfold(xt, k, dilation=dilation, padding=padding, stride=stride)  # [N, C*k*k, L]
    L = u.shape[-1]
    if order == "crs":
        want = u.permute(0, 2, 1).reshape(N * L, C * k * k)  # unfold's own order
    else:
        want = u.reshape(N, C, k, k, L).permute(0, 4, 2, 3, 1).reshape(N * L, k * k * C)
    assert y.shape == tuple(want.shape)
    assert np.array_equal(y.astype(np.float32), want.numpy())


def test_dilated_window_spot_values():
    """Tap (r, s) of output pixel (ho, wo) reads in[ho*stride + r*dilation - pad, wo*stride + s*dilation - pad]."""
    N, H, Wd, C = 1, 10, 12, 3
    x = (np.arange(N * H * Wd * C, dtype=np.uint32) + 1).reshape(N, H, Wd, C)
    k, stride, padding, dil = 3, 2, 2, 2
    Ho, Wo = (H + 2 * padding - dil * (k - 1) - 1) // stride + 1, (Wd + 2 * padding - dil * (k - 1) - 1) // stride + 1
    y = oracle.window(x, k, k, stride, padding, dilation=dil, order="rsc").reshape(Ho, Wo, k, k, C)
    z = oracle.window(x, k, k, stride, padding, dilation=dil, order="crs").reshape(Ho, Wo, C, k, k)
    for ho, wo, r, s_, c in [(0, 0, 0, 0, 0), (1, 2, 2, 1, 2), (Ho - 1, Wo - 1, 2, 2, 1), (2, 3, 1, 1, 0)]:
        h, w = ho * stride + r * dil - padding, wo * stride + s_ * dil - padding
        want = x[0, h, w, c] if 0 <= h < H and 0 <= w < Wd else 0
        assert y[ho, wo, r, s_, c] == want and z[ho, wo, c, r, s_] == want


# ---------------------------------------------------------------------------
# the generic load/store statement
# ---------------------------------------------------------------------------
def _python_stmt(dst, bounds, load, store, guarded, fill):
    Cs, bs = store
    for i in itertools.product(*[range(b) for b in bounds]):
        sidx = tuple(int(bs[d] + sum(Cs[d][k] * i[k] for k in range(len(i)))) for d in range(dst.ndim))
        if load is None:
            dst[sidx] = fill
            continue
        src, Cl, bl = load
        lidx = tuple(int(bl[d] + sum(Cl[d][k] * i[k] for k in range(len(i)))) for d in range(src.ndim))
        inside = all(0 <= v < n for v, n in zip(lidx, src.shape))
        assert inside or guarded
        dst[sidx] = src[lidx] if inside else fill


def test_affine_stmt_against_python_loops():
    for trial in range(30):
        n = int(rng.integers(1, 4))
        bounds = [int(rng.integers(1, 5)) for _ in range(n)]
        # an injective store: dst dims = loops, permuted, with offsets
        order = list(rng.permutation(n))
        offs = [int(rng.integers(0, 3)) for _ in range(n)]
        dshape = [bounds[order[d]] + offs[d] + int(rng.integers(0, 2)) for d in range(n)]
        Cs = [[1 if k == order[d] else 0 for k in range(n)] for d in range(n)]
        m = int(rng.integers(1, 4))
        Cl = [[int(rng.integers(-2, 3)) for _ in range(n)] for _ in range(m)]
        bl = [int(rng.integers(-1, 3)) for _ in range(m)]
        src = rand_u([int(rng.integers(3, 9)) for _ in range(m)], np.uint32)
        a = np.full(dshape, 0xDEAD, dtype=np.uint32)
        b = a.copy()
        oracle.affine_stmt(a, bounds, (src, Cl, bl), (Cs, offs), guarded=True, fill=77)
        _python_stmt(b, bounds, (src, Cl, bl), (Cs, offs), True, 77)
        assert np.array_equal(a, b), trial


def test_affine_stmt_refuses_an_unguarded_escape_and_fills_constants():
    src = rand_u((4,), np.uint16)
    dst = np.zeros((4,), np.uint16)
    with pytest.raises(ValueError):
        oracle.affine_stmt(dst, [4], (src, [[1]], [1]), ([[1]], [0]), guarded=False)
    oracle.affine_stmt(dst, [4], None, ([[1]], [0]), fill=0xBEEF)
    assert (dst == 0xBEEF).all()


def test_operator_families_as_load_store_pairs():
    """Each operator written out in the paper's form t_s[C_s i + b_s] = t_l[C_l i + b_l]
    gives what the operator's own loop nest gives (ties the generic statement to the rest)."""
    x = rand_u((4, 6, 5), np.uint32)
    # transpose(2,0,1): loops = output index (o0,o1,o2); load x[o1,o2,o0]
    y = np.zeros((5, 4, 6), np.uint32)
    oracle.affine_stmt(y, [5, 4, 6], (x, [[0, 1, 0], [0, 0, 1], [1, 0, 0]], [0, 0, 0]), (np.eye(3, dtype=int).tolist(), [0, 0, 0]))
    assert np.array_equal(y, oracle.transpose(x, [2, 0, 1]))
    # strided slice [1:4:2, :, 0:5:3]
    y = np.zeros((2, 6, 2), np.uint32)
    oracle.affine_stmt(y, [2, 6, 2], (x, [[2, 0, 0], [0, 1, 0], [0, 0, 3]], [1, 0, 0]), (np.eye(3, dtype=int).tolist(), [0, 0, 0]))
    assert np.array_equal(y, oracle.slice_(x, [1, 0, 0], [4, 6, 5], [2, 1, 3]))
    # pad by (1,2) on the middle axis as one guarded statement
    y = np.full((4, 9, 5), 9, np.uint32)
    oracle.affine_stmt(y, [4, 9, 5], (x, np.eye(3, dtype=int).tolist(), [0, -1, 0]), (np.eye(3, dtype=int).tolist(), [0, 0, 0]), guarded=True, fill=0)
    assert np.array_equal(y, oracle.pad(x, [0, 1, 0], [0, 2, 0]))
    # reshape [4,6,5] -> [8,15] over the common refinement (a<4, b<2, c<3, d<5)
    y = np.zeros((8, 15), np.uint32)
    oracle.affine_stmt(
        y, [4, 2, 3, 5], (x, [[1, 0, 0, 0], [0, 3, 1, 0], [0, 0, 0, 1]], [0, 0, 0]), ([[2, 1, 0, 0], [0, 0, 5, 1]], [0, 0])
    )
    assert np.array_equal(y, oracle.reshape(x, [8, 15]))
    # 3x3 window, stride 1, pad 1 as ONE guarded statement over (n,ho,wo,r,s,c)
    img = rand_u((2, 5, 4, 3), np.uint32)
    N, H, Wd, C = img.shape
    y = np.full((N * H * Wd, 9 * C), 5, np.uint32)
    Cl = [[1, 0, 0, 0, 0, 0], [0, 1, 0, 1, 0, 0], [0, 0, 1, 0, 1, 0], [0, 0, 0, 0, 0, 1]]
    Cs = [[H * Wd, Wd, 1, 0, 0, 0], [0, 0, 0, 3 * C, C, 1]]
    oracle.affine_stmt(y, [N, H, Wd, 3, 3, C], (img, Cl, [0, -1, -1, 0]), (Cs, [0, 0]), guarded=True, fill=0)
    assert np.array_equal(y, oracle.window(img, 3, 3, 1, 1))


# ---------------------------------------------------------------------------
# tile, repeat, split (the broadcast and cutting operators Section 2.1 names)
# ---------------------------------------------------------------------------
def test_tile_matches_numpy_and_counts_every_element():
    x = rand_u((3, 4, 5))
    reps = [2, 1, 3]
    y = oracle.tile(x, reps)
    assert y.shape == (6, 4, 15)
    assert np.array_equal(y, np.tile(x, reps))
    # each copy, cut back out by slicing, is the input; every value appears prod(reps) times as often
    for r0 in range(2):
        for r2 in range(3):
            part = oracle.slice_(y, [3 * r0, 0, 5 * r2], [3 * r0 + 3, 4, 5 * r2 + 5], [1, 1, 1])
            assert np.array_equal(part, x)
    vals, counts = np.unique(x, return_counts=True)
    vals_y, counts_y = np.unique(y, return_counts=True)
    assert np.array_equal(vals, vals_y) and np.array_equal(counts_y, 6 * counts)
    assert np.array_equal(oracle.tile(x, [1, 1, 1]), x)
    with pytest.raises(ValueError):
        oracle.tile(x, [1, 0, 1])


def test_repeat_matches_numpy_and_differs_from_tile():
    x = rand_u((3, 4, 5))
    for axis, count in ((0, 2), (1, 3), (2, 4)):
        y = oracle.repeat(x, axis, count)
        assert np.array_equal(y, np.repeat(x, count, axis=axis))
        # picking every count-th element along the axis, from any phase, gives the input back
        for phase in range(count):
            start = [0, 0, 0]
            start[axis] = phase
            assert np.array_equal(oracle.slice_(y, start, list(y.shape), [count if d == axis else 1 for d in range(3)]), x)
    # on the flat index of a rank-1 tensor: out[k] = in[k div count], not in[k mod n]
    v = np.arange(1, 6, dtype=np.uint16)
    assert oracle.repeat(v, 0, 3).tolist() == [1, 1, 1, 2, 2, 2, 3, 3, 3, 4, 4, 4, 5, 5, 5]
    assert oracle.tile(v, [3]).tolist() == [1, 2, 3, 4, 5] * 3
    assert np.array_equal(oracle.repeat(x, 1, 1), x)


def test_split_parts_match_numpy_and_join_back():
    x = rand_u((4, 9, 3))
    sizes = [2, 0, 3, 4]
    parts = [oracle.split_part(x, 1, sizes, k) for k in range(4)]
    want = np.split(x, np.cumsum(sizes)[:-1], axis=1)
    for got, w in zip(parts, want):
        assert got.shape == w.shape and np.array_equal(got, w)
    assert np.array_equal(oracle.concat(parts, 1), x)  # concat is the inverse of split
    with pytest.raises(ValueError):
        oracle.split_part(x, 1, [2, 3], 0)  # sizes do not add up to the extent


def test_broadcast_and_split_as_load_store_pairs():
    """tile, repeat and split written in the paper's form agree with the operators' own loop nests."""
    x = rand_u((3, 4), np.uint32)
    # tile(2, 3): loops (r0, i0, r1, i1); the load ignores the repetition loops
    y = np.zeros((6, 12), np.uint32)
    oracle.affine_stmt(y, [2, 3, 3, 4], (x, [[0, 1, 0, 0], [0, 0, 0, 1]], [0, 0]), ([[3, 1, 0, 0], [0, 0, 4, 1]], [0, 0]))
    assert np.array_equal(y, oracle.tile(x, [2, 3]))
    # repeat(axis 1, 3): loops (i0, i1, j)
    y = np.zeros((3, 12), np.uint32)
    oracle.affine_stmt(y, [3, 4, 3], (x, [[1, 0, 0], [0, 1, 0]], [0, 0]), ([[1, 0, 0], [0, 3, 1]], [0, 0]))
    assert np.array_equal(y, oracle.repeat(x, 1, 3))
    # split(axis 1, [1, 3]) part 1: loops = part index, load offset 1
    y = np.zeros((3, 3), np.uint32)
    oracle.affine_stmt(y, [3, 3], (x, [[1, 0], [0, 1]], [0, 1]), ([[1, 0], [0, 1]], [0, 0]))
    assert np.array_equal(y, oracle.split_part(x, 1, [1, 3], 1))


# ---------------------------------------------------------------------------
# brute force on tiny random chains
# ---------------------------------------------------------------------------
def _python_chain(chain, inputs):
    ts = [np.asarray(x) for x in inputs]
    for op in chain.ops:
        k = op["kind"]
        if k == "reshape":
            t = ts[op["src"]].reshape(op["shape"])
        elif k == "transpose":
            t = np.transpose(ts[op["src"]], op["perm"])
        elif k == "slice":
            t = ts[op["src"]][tuple(slice(a, b, s) for a, b, s in zip(op["start"], op["stop"], op["step"]))]
        elif k == "concat":
            t = np.concatenate([ts[s] for s in op["srcs"]], op["axis"])
        elif k == "pad":
            t = np.pad(ts[op["src"]], list(zip(op["lo"], op["hi"])))
        elif k == "tile":
            t = np.tile(ts[op["src"]], op["reps"])
        elif k == "repeat":
            t = np.repeat(ts[op["src"]], op["count"], axis=op["axis"])
        elif k == "split":
            t = np.split(ts[op["src"]], np.cumsum(op["sizes"])[:-1], axis=op["axis"])[op["part"]]
        ts.append(np.ascontiguousarray(t))
    return ts[-1]


def test_random_tiny_chains_against_numpy():
    r = np.random.default_rng(2002)
    for trial in range(150):
        chain = random_chain(r)
        xs = W.make_index_tagged_inputs(chain)
        xs = [x + np.uint32(1) for x in xs]  # keep 0 for padding
        got = oracle.run_chain(chain, xs)
        want = _python_chain(chain, xs)
        assert got.shape == want.shape, (trial, chain.ops)
        assert np.array_equal(got, want), (trial, chain.ops)
