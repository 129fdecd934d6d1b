"""Random tiny chains of layout operators (plain data; used by CPU and GPU tests)."""
import numpy as np

from paper_2002_12798_b200 import workloads as W


def random_chain(r, n_ops=4, max_extent=5, max_rank=4):
    """A random chain of <= n_ops operators over one or two tiny inputs."""
    rank = int(r.integers(1, max_rank + 1))
    shape = [int(r.integers(1, max_extent + 1)) for _ in range(rank)]
    inputs = [shape]
    ops = []
    cur, cur_shape = 0, list(shape)
    for _ in range(n_ops):
        kind = r.choice(["reshape", "transpose", "slice", "pad", "concat", "tile", "repeat", "split"])
        tid = len(inputs) + len(ops)
        if kind == "reshape":
            n = int(np.prod(cur_shape))
            facs = []
            rem = n
            for _ in range(int(r.integers(1, 4))):
                divs = [d for d in range(1, rem + 1) if rem % d == 0]
                f = int(r.choice(divs))
                facs.append(f)
                rem //= f
            facs.append(rem)
            r.shuffle(facs)
            ops.append({"kind": "reshape", "src": cur, "shape": [int(f) for f in facs]})
            cur_shape = [int(f) for f in facs]
        elif kind == "transpose":
            perm = [int(p) for p in r.permutation(len(cur_shape))]
            ops.append({"kind": "transpose", "src": cur, "perm": perm})
            cur_shape = [cur_shape[p] for p in perm]
        elif kind == "slice":
            start, stop, step = [], [], []
            for n in cur_shape:
                a = int(r.integers(0, n))
                b = int(r.integers(a + 1, n + 1))
                s = int(r.integers(1, 3))
                start.append(a), stop.append(b), step.append(s)
            ops.append({"kind": "slice", "src": cur, "start": start, "stop": stop, "step": step})
            cur_shape = [-(-(b - a) // s) for a, b, s in zip(start, stop, step)]
        elif kind == "pad":
            lo = [int(r.integers(0, 2)) for _ in cur_shape]
            hi = [int(r.integers(0, 2)) for _ in cur_shape]
            ops.append({"kind": "pad", "src": cur, "lo": lo, "hi": hi})
            cur_shape = [a + n + b for a, n, b in zip(lo, cur_shape, hi)]
        elif kind == "tile":
            reps = [int(r.integers(1, 3)) for _ in cur_shape]
            ops.append({"kind": "tile", "src": cur, "reps": reps})
            cur_shape = [a * n for a, n in zip(reps, cur_shape)]
        elif kind == "repeat":
            axis = int(r.integers(0, len(cur_shape)))
            count = int(r.integers(1, 4))
            ops.append({"kind": "repeat", "src": cur, "axis": axis, "count": count})
            cur_shape = list(cur_shape)
            cur_shape[axis] *= count
        elif kind == "split":
            axis = int(r.integers(0, len(cur_shape)))
            n = cur_shape[axis]
            cut = sorted(int(c) for c in r.integers(0, n + 1, size=2))
            sizes = [cut[0], cut[1] - cut[0], n - cut[1]]
            part = int(r.choice([k for k in range(3) if sizes[k] > 0]))
            ops.append({"kind": "split", "src": cur, "axis": axis, "sizes": sizes, "part": part})
            cur_shape = list(cur_shape)
            cur_shape[axis] = sizes[part]
        else:  # concat the current tensor with itself or with the first input when shapes allow
            axis = int(r.integers(0, len(cur_shape)))
            other = cur
            ops.append({"kind": "concat", "srcs": [cur, other], "axis": axis})
            cur_shape = list(cur_shape)
            cur_shape[axis] *= 2
        cur = tid
        if int(np.prod(cur_shape)) > 4000:
            break
    return W.Chain(name="random", dtype="fp32", inputs=inputs, ops=ops, values="raw")
