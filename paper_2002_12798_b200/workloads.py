"""Seeded synthetic workloads: chain descriptions and input bytes.

This module is plain data plus a random-number recipe.  It performs none of the
method's arithmetic (no index maps, no shape inference, no composition): a
chain is a list of operator *parameters*, and each consumer (the CPU oracle,
the CUDA library's builder) interprets them with its own code.

Chain format
------------
``Chain.inputs``  shapes of the external input tensors; they get tensor ids
                  0 .. n_inputs-1.
``Chain.ops``     list of dicts; op number k defines tensor id n_inputs + k.
                  The last op's tensor is the chain's output.  Kinds:

  {"kind": "reshape",   "src": t, "shape": [...]}
  {"kind": "transpose", "src": t, "perm": [...]}        out.shape[d] = in.shape[perm[d]]
  {"kind": "slice",     "src": t, "start": [...], "stop": [...], "step": [...]}
  {"kind": "concat",    "srcs": [t0, t1, ...], "axis": a}
  {"kind": "pad",       "src": t, "lo": [...], "hi": [...]}          zero fill
  {"kind": "window",    "src": t, "kh":, "kw":, "stride":, "pad":}   NHWC im2col, column order (r, s, c);
                        optional "dilation": d (taps d pixels apart), "order": "rsc" | "crs" (column order)
  {"kind": "tile",      "src": t, "reps": [...]}                     the whole tensor reps[d] times along axis d
  {"kind": "repeat",    "src": t, "axis": a, "count": c}             every element c times in a row along axis a
  {"kind": "split",     "src": t, "axis": a, "sizes": [...], "part": k}   part k of t cut along axis a
  {"kind": "stmts",     "shape": [...], "stmts": [ {...}, ... ]}     raw load/store pairs in the paper's form:
        {"bounds": [...], "load": None | (tensor, C rows, b), "store": (C rows, b),
         "guarded": bool, "fill": int}

Values are opaque bit patterns to the method; the recipes below only make them
look like the activations of CNN / Transformer inference (the paper evaluates
on Parallel WaveNet and ResNet-50, whose tensors are not available; these
shapes stand in for them).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

ELEM_SIZE = {"fp32": 4, "bf16": 2, "fp16": 2, "u8": 1, "u64": 8}
RAW_DTYPE = {1: np.uint8, 2: np.uint16, 4: np.uint32, 8: np.uint64}
BASE_SEED = 12798


@dataclass
class Chain:
    name: str
    dtype: str
    inputs: list
    ops: list
    values: str = "normal"  # "normal" | "uniform_pm1" | "uniform_int20"
    seed: int = BASE_SEED
    note: str = ""
    meta: dict = field(default_factory=dict)

    @property
    def elem_size(self) -> int:
        return ELEM_SIZE[self.dtype]

    @property
    def n_inputs(self) -> int:
        return len(self.inputs)


# ----------------------------------------------------------------------------
# value recipes (bit patterns of the stated dtype, returned as unsigned ints)
# ----------------------------------------------------------------------------
def _f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even truncation of fp32 to its upper 16 bits."""
    u = x.astype(np.float32).view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def make_values(n: int, dtype: str, values: str, rng: np.random.Generator) -> np.ndarray:
    """n seeded elements of `dtype` as raw unsigned integers of the same width."""
    if values == "raw" or dtype in ("u8", "u64"):
        es = ELEM_SIZE[dtype]
        return rng.integers(0, 1 << (8 * min(es, 4)), size=n, dtype=np.uint64).astype(RAW_DTYPE[es])
    if values == "uniform_int20":
        f = rng.integers(0, 1 << 20, size=n, dtype=np.int64).astype(np.float32)
    elif values == "uniform_pm1":
        f = rng.random(size=n, dtype=np.float32) * np.float32(2.0) - np.float32(1.0)
    elif values == "normal":
        f = rng.standard_normal(size=n, dtype=np.float32)
    else:
        raise ValueError(values)
    if dtype == "fp32":
        return f.view(np.uint32)
    if dtype == "bf16":
        return _f32_to_bf16_bits(f)
    if dtype == "fp16":
        return f.astype(np.float16).view(np.uint16)
    raise ValueError(dtype)


def make_inputs(chain: Chain, seed: int | None = None) -> list:
    """One raw-bits array per external input, shaped like the input."""
    rng = np.random.default_rng(chain.seed if seed is None else seed)
    out = []
    for shape in chain.inputs:
        n = int(np.prod(shape, dtype=np.int64))
        out.append(make_values(n, chain.dtype, chain.values, rng).reshape(shape))
    return out


def make_index_tagged_inputs(chain: Chain, part: int = 0) -> list:
    """Inputs whose every element holds (a slice of) its own identity.

    Element k of input q carries the number q * 2**40 + k; 4-byte (or wider)
    elements hold its low 32 bits (``part`` 0) or the next 32 bits
    (``part`` 1); 2-byte elements hold bits 16*part .. 16*part+15, 1-byte
    elements bits 8*part ...  Copying such inputs through a chain turns the
    output into the chain's source-index map.
    """
    es = chain.elem_size
    bits = 8 * min(es, 4)
    out = []
    for q, shape in enumerate(chain.inputs):
        n = int(np.prod(shape, dtype=np.int64))
        tag = np.arange(n, dtype=np.uint64) + (np.uint64(q) << np.uint64(40))
        part_bits = (tag >> np.uint64(bits * part)) & np.uint64((1 << bits) - 1)
        out.append(part_bits.astype(RAW_DTYPE[es]).reshape(shape))
    return out


# ----------------------------------------------------------------------------
# the five configurations (and reduced-size versions with the same structure)
# ----------------------------------------------------------------------------
def c1_small_chain() -> Chain:
    """fp32 [64,128]: reshape -> transpose(2,0,1) -> slice -> reshape [64,48]."""
    return Chain(
        name="c1_small_chain",
        dtype="fp32",
        inputs=[[64, 128]],
        ops=[
            {"kind": "reshape", "src": 0, "shape": [8, 8, 128]},
            {"kind": "transpose", "src": 1, "perm": [2, 0, 1]},
            {"kind": "slice", "src": 2, "start": [0, 0, 1], "stop": [128, 8, 7], "step": [2, 1, 1]},
            {"kind": "reshape", "src": 3, "shape": [64, 48]},
        ],
        values="uniform_int20",
        seed=BASE_SEED + 1,
    )


def c2_nchw_to_nhwc(N=32, C=256, H=56, W=56, dtype="bf16") -> Chain:
    return Chain(
        name="c2_nchw_to_nhwc",
        dtype=dtype,
        inputs=[[N, C, H, W]],
        ops=[{"kind": "transpose", "src": 0, "perm": [0, 2, 3, 1]}],
        values="normal",
        seed=BASE_SEED + 2,
    )


def c2_nhwc_to_nchw(N=32, C=256, H=56, W=56, dtype="bf16") -> Chain:
    return Chain(
        name="c2_nhwc_to_nchw",
        dtype=dtype,
        inputs=[[N, H, W, C]],
        ops=[{"kind": "transpose", "src": 0, "perm": [0, 3, 1, 2]}],
        values="normal",
        seed=BASE_SEED + 2,
    )


def c3_head_split(B=16, S=2048, heads=32, D=128, keep=1536, dtype="bf16") -> Chain:
    """Two [B,S,heads*D] tensors: each reshaped to [B,S,heads,D], moved to
    [B,heads,S,D], cut to the first `keep` positions; then joined on S."""
    ops = []
    outs = []
    for q in range(2):
        base = 2 + len(ops)
        ops.append({"kind": "reshape", "src": q, "shape": [B, S, heads, D]})
        ops.append({"kind": "transpose", "src": base, "perm": [0, 2, 1, 3]})
        ops.append(
            {
                "kind": "slice",
                "src": base + 1,
                "start": [0, 0, 0, 0],
                "stop": [B, heads, keep, D],
                "step": [1, 1, 1, 1],
            }
        )
        outs.append(base + 2)
    ops.append({"kind": "concat", "srcs": outs, "axis": 2})
    return Chain(
        name="c3_head_split",
        dtype=dtype,
        inputs=[[B, S, heads * D], [B, S, heads * D]],
        ops=ops,
        values="normal",
        seed=BASE_SEED + 3,
    )


def c3_head_merge(B=16, S=3072, heads=32, D=128, dtype="bf16") -> Chain:
    """The inverse direction: [B,heads,S,D] -> [B,S,heads,D] -> [B,S,heads*D]."""
    return Chain(
        name="c3_head_merge",
        dtype=dtype,
        inputs=[[B, heads, S, D]],
        ops=[
            {"kind": "transpose", "src": 0, "perm": [0, 2, 1, 3]},
            {"kind": "reshape", "src": 1, "shape": [B, S, heads * D]},
        ],
        values="normal",
        seed=BASE_SEED + 3,
    )


def c4_inception_concat(N=64, channels=(64, 96, 128, 32), H=28, W=28, dtype="fp16") -> Chain:
    """Four NCHW branches, each zero-padded by 1 on H and W, joined on C, to NHWC."""
    nb = len(channels)
    ops = []
    for q in range(nb):
        ops.append({"kind": "pad", "src": q, "lo": [0, 0, 1, 1], "hi": [0, 0, 1, 1]})
    ops.append({"kind": "concat", "srcs": [nb + q for q in range(nb)], "axis": 1})
    ops.append({"kind": "transpose", "src": 2 * nb, "perm": [0, 2, 3, 1]})
    return Chain(
        name="c4_inception_concat",
        dtype=dtype,
        inputs=[[N, c, H, W] for c in channels],
        ops=ops,
        values="uniform_pm1",
        seed=BASE_SEED + 4,
    )


def c5_im2col(N=64, H=56, W=56, C=128, k=3, stride=1, pad=1, dtype="fp16", dilation=1, order="rsc") -> Chain:
    op = {"kind": "window", "src": 0, "kh": k, "kw": k, "stride": stride, "pad": pad}
    if dilation != 1:
        op["dilation"] = dilation
    if order != "rsc":
        op["order"] = order
    return Chain(
        name="c5_im2col",
        dtype=dtype,
        inputs=[[N, H, W, C]],
        ops=[op],
        values="uniform_pm1",
        seed=BASE_SEED + 5,
    )


def upsample_nhwc(N=32, H=56, W=56, C=256, factor=2, dtype="fp16") -> Chain:
    """Nearest-neighbour upsampling of NHWC activations: every pixel `factor` times along H and along W."""
    return Chain(
        name="upsample_nhwc",
        dtype=dtype,
        inputs=[[N, H, W, C]],
        ops=[
            {"kind": "repeat", "src": 0, "axis": 1, "count": factor},
            {"kind": "repeat", "src": 1, "axis": 2, "count": factor},
        ],
        values="uniform_pm1",
        seed=BASE_SEED + 6,
    )


def qkv_split(B=16, S=2048, heads=32, D=128, part=0, dtype="bf16") -> Chain:
    """The output [B,S,3*heads*D] of a fused QKV projection cut into three on the last axis; part `part`
    reshaped to [B,S,heads,D] and moved to [B,heads,S,D]."""
    hd = heads * D
    return Chain(
        name="qkv_split_%d" % part,
        dtype=dtype,
        inputs=[[B, S, 3 * hd]],
        ops=[
            {"kind": "split", "src": 0, "axis": 2, "sizes": [hd, hd, hd], "part": part},
            {"kind": "reshape", "src": 1, "shape": [B, S, heads, D]},
            {"kind": "transpose", "src": 2, "perm": [0, 2, 1, 3]},
        ],
        values="normal",
        seed=BASE_SEED + 7,
    )


def qkv_split_all(B=16, S=2048, heads=32, D=128, dtype="bf16") -> Chain:
    """The same cut with all three parts in ONE chain; `meta["outputs"]` names the three results (tensor numbers)."""
    hd = heads * D
    ops = []
    outs = []
    for part in range(3):
        base = 1 + len(ops)
        ops.append({"kind": "split", "src": 0, "axis": 2, "sizes": [hd, hd, hd], "part": part})
        ops.append({"kind": "reshape", "src": base, "shape": [B, S, heads, D]})
        ops.append({"kind": "transpose", "src": base + 1, "perm": [0, 2, 1, 3]})
        outs.append(base + 2)
    return Chain(name="qkv_split_all", dtype=dtype, inputs=[[B, S, 3 * hd]], ops=ops, values="normal", seed=BASE_SEED + 7,
                 meta={"outputs": outs})


def full_configs() -> dict:
    """The configurations at the sizes the benchmark quotes."""
    return {
        "c1": c1_small_chain(),
        "c2_fwd": c2_nchw_to_nhwc(),
        "c2_inv": c2_nhwc_to_nchw(),
        "c3": c3_head_split(),
        "c3_merge": c3_head_merge(),
        "c4": c4_inception_concat(),
        "c5": c5_im2col(),
    }


def reduced_configs() -> dict:
    """Same structure, sizes the oracle finishes in a second or two, still
    spanning several tiles with ragged tails."""
    return {
        "c1": c1_small_chain(),
        "c2_fwd": c2_nchw_to_nhwc(N=3, C=72, H=13, W=11),
        "c2_inv": c2_nhwc_to_nchw(N=3, C=72, H=13, W=11),
        "c2_fwd_mid": c2_nchw_to_nhwc(N=2, C=256, H=56, W=56),
        "c2_inv_mid": c2_nhwc_to_nchw(N=2, C=256, H=56, W=56),
        "c2_fwd_rag": c2_nchw_to_nhwc(N=2, C=72, H=13, W=8),
        "c2_inv_rag": c2_nhwc_to_nchw(N=2, C=72, H=13, W=8),
        "c2_fwd_f32": c2_nchw_to_nhwc(N=2, C=36, H=13, W=12, dtype="fp32"),
        "c2_inv_u8": c2_nhwc_to_nchw(N=2, C=80, H=14, W=8, dtype="u8"),
        "c2_fwd_u64": c2_nchw_to_nhwc(N=2, C=34, H=5, W=6, dtype="u64"),
        "c2_fwd_odd_f32": c2_nchw_to_nhwc(N=2, C=37, H=7, W=9, dtype="fp32"),
        "c2_inv_odd_u8": c2_nhwc_to_nchw(N=2, C=64, H=11, W=13, dtype="u8"),
        "c2_inv_odd_f32": c2_nhwc_to_nchw(N=2, C=36, H=7, W=9, dtype="fp32"),
        "c2_inv_odd_big": c2_nhwc_to_nchw(N=2, C=256, H=27, W=27),
        "c2_fwd_odd_big": c2_nchw_to_nhwc(N=2, C=256, H=27, W=27),
        "c2_fwd_odd_gather": c2_nchw_to_nhwc(N=2, C=255, H=27, W=27),
        # misaligned destination rows: shorter than a tile, just longer than one, of 4- and 1-byte elements, and
        # with a gap after every row (so that a row does not continue where the one before ends)
        "c2_inv_7x7": c2_nhwc_to_nchw(N=3, C=136, H=7, W=7),
        "c2_inv_67": c2_nhwc_to_nchw(N=2, C=40, H=67, W=1),
        "c2_inv_65": c2_nhwc_to_nchw(N=2, C=24, H=5, W=13),
        "c2_inv_33_f32": c2_nhwc_to_nchw(N=2, C=20, H=3, W=11, dtype="fp32"),
        "c2_inv_131_u8": c2_nhwc_to_nchw(N=2, C=48, H=131, W=1, dtype="u8"),
        "c2_inv_gap": Chain(
            name="c2_inv_gap", dtype="bf16", inputs=[[2, 5, 25, 48]],
            ops=[{"kind": "transpose", "src": 0, "perm": [0, 3, 1, 2]},
                 {"kind": "pad", "src": 1, "lo": [0, 0, 0, 0], "hi": [0, 0, 0, 2]}],
            values="normal", seed=BASE_SEED + 2,
        ),
        # panels that are contiguous in the destination (the flat-destination transpose): large panels on blocks of
        # 512 threads, a source that is a window of a larger tensor (two strides along the pixels), two batch loops,
        # a last panel with fewer channels than the others, 4-byte elements
        "c2_inv_flat_big": c2_nhwc_to_nchw(N=20, C=256, H=27, W=27),
        "c2_inv_flat_big_f32": c2_nhwc_to_nchw(N=19, C=136, H=19, W=21, dtype="fp32"),
        "c2_inv_flat_window": Chain(
            name="c2_inv_flat_window", dtype="bf16", inputs=[[3, 9, 12, 104]],
            ops=[{"kind": "slice", "src": 0, "start": [0, 1, 2, 0], "stop": [3, 8, 9, 104], "step": [1, 1, 1, 1]},
                 {"kind": "transpose", "src": 1, "perm": [0, 3, 1, 2]}],
            values="normal", seed=BASE_SEED + 2,
        ),
        "c2_inv_flat_5d": Chain(
            name="c2_inv_flat_5d", dtype="fp16", inputs=[[2, 4, 5, 7, 168]],
            ops=[{"kind": "slice", "src": 0, "start": [0, 1, 0, 0, 0], "stop": [2, 4, 5, 7, 168], "step": [1, 1, 1, 1, 1]},
                 {"kind": "transpose", "src": 1, "perm": [0, 1, 4, 2, 3]}],
            values="normal", seed=BASE_SEED + 2,
        ),
        "c2_fwd_odd_u8": c2_nchw_to_nhwc(N=2, C=64, H=11, W=13, dtype="u8"),
        "c2_fwd_odd_f32b": c2_nchw_to_nhwc(N=2, C=36, H=7, W=9, dtype="fp32"),
        "c2_fwd_narrow": c2_nchw_to_nhwc(N=2, C=72, H=14, W=14),
        "c2_inv_narrow": c2_nhwc_to_nchw(N=2, C=68, H=14, W=14),
        # rows aligned to 4 bytes only, on both sides: 4-byte units
        "c2_fwd_both4": c2_nchw_to_nhwc(N=2, C=70, H=6, W=9),
        "c2_inv_both4": c2_nhwc_to_nchw(N=2, C=70, H=6, W=9),
        # 16-byte transposes whose extent along the destination run leaves at most half a tile (remainder pieces on
        # the 64-byte tile), or is that short altogether; several tiles along the other index, evenly stepped
        "c2_fwd_rem": c2_nchw_to_nhwc(N=2, C=96, H=20, W=26),
        "c2_fwd_rem_f32": c2_nchw_to_nhwc(N=2, C=40, H=12, W=23, dtype="fp32"),
        "c2_fwd_rem_u8": c2_nchw_to_nhwc(N=2, C=160, H=16, W=37, dtype="u8"),
        "c2_fwd_rem_u64": c2_nchw_to_nhwc(N=2, C=20, H=10, W=53, dtype="u64"),
        "c2_fwd_short": c2_nchw_to_nhwc(N=2, C=24, H=20, W=26),
        "c2_inv_rem": c2_nhwc_to_nchw(N=2, C=280, H=8, W=12),
        # 16-byte transposes that are short along the source run (64 or 32 channels in NHWC): wide, flat tiles
        "c2_inv_c64": c2_nhwc_to_nchw(N=2, C=64, H=24, W=20),
        "c2_inv_c48": c2_nhwc_to_nchw(N=2, C=48, H=24, W=20),
        "c2_inv_c32_f32": c2_nhwc_to_nchw(N=2, C=32, H=12, W=23, dtype="fp32"),
        "c2_inv_c64_f32": c2_nhwc_to_nchw(N=2, C=64, H=12, W=23, dtype="fp32"),
        "c2_inv_c24_u64": c2_nhwc_to_nchw(N=2, C=24, H=10, W=27, dtype="u64"),
        "c2_fwd_hw64": c2_nchw_to_nhwc(N=2, C=200, H=8, W=8),
        "c3": c3_head_split(B=2, S=80, heads=3, D=128, keep=50),
        "c3_odd": c3_head_split(B=2, S=33, heads=5, D=24, keep=17),
        "c3_merge": c3_head_merge(B=2, S=70, heads=3, D=128),
        "c4": c4_inception_concat(N=2, channels=(64, 96, 128, 32), H=28, W=28),
        "c4_odd": c4_inception_concat(N=3, channels=(8, 24, 40, 16), H=7, W=9),
        "c5": c5_im2col(N=2, H=14, W=12, C=128),
        "c5_odd": c5_im2col(N=2, H=9, W=7, C=24, k=3, stride=2, pad=1),
        "c5_5x5": c5_im2col(N=2, H=10, W=9, C=24, k=5, stride=1, pad=2),
        "c5_5x5_wide": c5_im2col(N=1, H=12, W=11, C=128, k=5, stride=2, pad=2),
        # dilated taps and the (c, r, s) column order of NCHW im2col
        "c5_dil2": c5_im2col(N=2, H=13, W=11, C=128, k=3, stride=1, pad=2, dilation=2),
        "c5_dil3_s2": c5_im2col(N=2, H=14, W=15, C=24, k=3, stride=2, pad=3, dilation=3),
        "c5_crs": c5_im2col(N=2, H=10, W=12, C=64, k=3, stride=1, pad=1, order="crs"),
        "c5_crs_dil2_f32": c5_im2col(N=1, H=9, W=11, C=20, k=3, stride=2, pad=2, dilation=2, order="crs", dtype="fp32"),
    }
