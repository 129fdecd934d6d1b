"""Random raw load/store statements (the paper's form, arbitrary small integer C and b): whenever amap_compose
accepts a chain its map must reproduce the oracle's sequential execution; otherwise it must fail with one of its
documented codes.  Nothing here may crash."""
import numpy as np

from oracle import oracle
from paper_2002_12798_b200 import binding as B
from paper_2002_12798_b200 import workloads as W
from test_compose import eval_map

ALLOWED = {-2, -3, -4, -5, -9}  # not injective, out of bounds, undefined, overlap, unsupported


def _corner_range(C_row, b, bounds):
    lo = hi = b
    for c, n in zip(C_row, bounds):
        if c > 0:
            hi += c * (n - 1)
        else:
            lo += c * (n - 1)
    return lo, hi


def random_stmt_chain(r):
    """Tensors defined by one or two statements that together write every element once (boxes split along an
    axis, interleaved even/odd stores, two loops merged into one axis), with arbitrary small affine loads."""
    inputs = [[int(r.integers(2, 6)) for _ in range(int(r.integers(1, 3)))] for _ in range(int(r.integers(1, 3)))]
    shapes = [list(s) for s in inputs]
    ops = []
    for _ in range(int(r.integers(1, 4))):
        rank = int(r.integers(1, 4))
        shape = [int(r.integers(2, 6)) for _ in range(rank)]
        mode = r.choice(["whole", "split", "interleave", "merged"])
        boxes = []  # (bounds, Cs, bs)
        eye = [[1 if k == d else 0 for k in range(rank)] for d in range(rank)]
        if mode == "split":
            cut = int(r.integers(1, shape[0]))
            boxes.append(([cut] + shape[1:], eye, [0] * rank))
            boxes.append(([shape[0] - cut] + shape[1:], eye, [cut] + [0] * (rank - 1)))
        elif mode == "interleave":
            shape[0] = 2 * int(r.integers(1, 4))
            two = [[2 if (k == d == 0) else eye[d][k] for k in range(rank)] for d in range(rank)]
            boxes.append(([shape[0] // 2] + shape[1:], two, [0] * rank))
            boxes.append(([shape[0] // 2] + shape[1:], two, [1] + [0] * (rank - 1)))
        elif mode == "merged":  # axis 0 is fed by two loops (a mixed-radix pair), in a random loop order
            e_in = int(r.integers(2, 4))
            shape[0] = e_in * int(r.integers(1, 4))
            bounds = [shape[0] // e_in, e_in] + shape[1:]
            Cs = [[0] * (rank + 1) for _ in range(rank)]
            Cs[0][0], Cs[0][1] = e_in, 1
            for d in range(1, rank):
                Cs[d][d + 1] = 1
            boxes.append((bounds, Cs, [0] * rank))
        else:
            boxes.append((list(shape), eye, [0] * rank))
        stmts = []
        for bounds, Cs, bs in boxes:
            n = len(bounds)
            perm = [int(k) for k in r.permutation(n)]  # the loop order is arbitrary
            bounds = [bounds[k] for k in perm]
            Cs = [[row[k] for k in perm] for row in Cs]
            if r.random() < 0.1:
                load, guarded = None, False
            else:
                lt = int(r.integers(0, len(shapes)))
                Cl = [[int(r.integers(-1, 3)) for _ in range(n)] for _ in shapes[lt]]
                bl = [int(r.integers(-1, 3)) for _ in shapes[lt]]
                escapes = any(not (0 <= lo and hi < ext) for (lo, hi), ext in
                              zip((_corner_range(row, b0, bounds) for row, b0 in zip(Cl, bl)), shapes[lt]))
                guarded = escapes or bool(r.random() < 0.3)
                load = (lt, Cl, bl)
            stmts.append({"bounds": bounds, "load": load, "store": (Cs, bs), "guarded": guarded, "fill": 7})
        ops.append({"kind": "stmts", "shape": shape, "stmts": stmts})
        shapes.append(shape)
    return W.Chain(name="fuzz", dtype="fp32", inputs=inputs, ops=ops, values="raw")


def test_random_statement_chains():
    r = np.random.default_rng(20200229)
    accepted = refused = 0
    for trial in range(600):
        chain = random_stmt_chain(r)
        xs = [x + np.uint32(100) for x in W.make_index_tagged_inputs(chain)]
        try:
            m = B.compose_chain(chain)
        except B.AmapError as e:
            assert e.code in ALLOWED, (trial, e.code, chain.ops)
            refused += 1
            continue
        want = oracle.run_chain(chain, xs)  # must not refuse what the library accepted
        assert np.array_equal(eval_map(m, xs), want.reshape(-1)), (trial, chain.ops)
        m.plan(device=-1)  # and the planner's address replay must hold
        accepted += 1
    assert accepted >= 300, (accepted, refused)
