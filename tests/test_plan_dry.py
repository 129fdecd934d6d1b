"""Planner decisions on the CPU (dry plans: amap_plan with device = -1 makes no CUDA call).  The dry plan also
replays every descriptor's address arithmetic on the host, so a wrong table fails here, not on a GPU."""
import pytest

from paper_2002_12798_b200 import binding as B
from paper_2002_12798_b200 import workloads as W


def kernels(chain, **kw):
    st = B.compose_chain(chain).plan(device=-1, **kw).stats()
    return st["kernels"], st["n_launches"], st["n_stages"]


def test_full_configurations_each_run_as_one_launch():
    full = W.full_configs()
    assert kernels(full["c2_fwd"]) == ({"gather": 0, "copy": 0, "transpose": 1, "fill": 0}, 1, 1)
    assert kernels(full["c2_inv"]) == ({"gather": 0, "copy": 0, "transpose": 1, "fill": 0}, 1, 1)
    assert kernels(full["c3"]) == ({"gather": 0, "copy": 2, "transpose": 0, "fill": 0}, 1, 1)
    assert kernels(full["c4"]) == ({"gather": 0, "copy": 0, "transpose": 4, "fill": 4}, 1, 1)
    assert kernels(full["c5"]) == ({"gather": 0, "copy": 1, "transpose": 0, "fill": 0}, 1, 1)
    assert kernels(full["c1"])[0]["gather"] == 1  # a strided innermost load: element-wise gather


def test_forced_families():
    c2 = W.full_configs()["c2_fwd"]
    assert kernels(c2, force_kernel=B.KERNEL_GATHER)[0]["gather"] == 1
    assert kernels(c2, force_kernel=B.KERNEL_COPY)[0]["transpose"] == 0
    assert kernels(c2, pointer_align=2)[0]["transpose"] == 0  # no 16-byte promise: no vector kernels


@pytest.mark.parametrize(
    "shape,expect",
    [
        ((4, 256, 56, 56), "transpose"),  # 16-byte rows on both sides
        ((4, 256, 14, 14), "transpose"),  # 8-byte aligned rows: narrow units
        ((4, 254, 54, 54), "transpose"),  # 4-byte aligned
        ((4, 256, 27, 27), "transpose"),  # odd source rows, aligned destination rows: realigning kernel
        ((4, 255, 27, 27), "gather"),     # both sides misaligned: strip kernel
    ],
)
def test_transpose_family_by_alignment(shape, expect):
    n, c, h, w = shape
    k, launches, _ = kernels(W.c2_nchw_to_nhwc(N=n, C=c, H=h, W=w))
    assert k[expect] == 1 and launches == 1


def test_shifted_transpose_for_misaligned_destination_rows():
    k, _, _ = kernels(W.c2_nhwc_to_nchw(N=4, C=256, H=27, W=27))
    assert k["transpose"] == 1
    k, _, _ = kernels(W.c2_nhwc_to_nchw(N=4, C=255, H=27, W=27))  # source rows misaligned too
    assert k["gather"] == 1


def launch_of(chain):
    launches = B.compose_chain(chain).plan(device=-1).launches()
    assert len(launches) == 1
    return launches[0]


def test_transpose_kernel_per_shape():
    """NHWC -> NCHW: which of the transpose kernels a shape gets (amap_plan_launch_info), with the block size and
    the shared memory of the flat-destination kernel's panels."""
    inv = W.c2_nhwc_to_nchw
    L = launch_of(inv(N=32, C=256, H=56, W=56))  # rows of 6272 bytes, aligned on both sides
    assert (L["kernel"], L["access"], L["threads"], L["smem_bytes"]) == ("transpose", 16, 256, 0)
    # 35x35 maps: rows of 2450 bytes; a panel of all 1225 pixels by 32 channels is 78400 bytes, 9 panels per image
    L = launch_of(inv(N=64, C=288, H=35, W=35))
    assert (L["kernel"], L["threads"], L["smem_bytes"], L["n_blocks"]) == ("transpose_flat", 512, 78400, 64 * 9)
    # 14x14 maps: rows of 392 bytes; 32 channels make a panel of 12544 bytes (64 channels would pass 24 KB)
    L = launch_of(inv(N=64, C=1024, H=14, W=14))
    assert (L["kernel"], L["threads"], L["smem_bytes"], L["n_blocks"]) == ("transpose_flat", 256, 12544, 64 * 32)
    # 7x7 maps: rows of 98 bytes; 128 channels (256 bytes per pixel, the most a panel takes) make 12544 bytes
    L = launch_of(inv(N=64, C=2048, H=7, W=7))
    assert (L["kernel"], L["threads"], L["smem_bytes"], L["n_blocks"]) == ("transpose_flat", 256, 12544, 64 * 16)
    # 4-byte elements: 64 bytes of the source run are 16 channels
    L = launch_of(inv(N=19, C=136, H=19, W=21, dtype="fp32"))
    assert (L["kernel"], L["threads"], L["smem_bytes"], L["n_blocks"]) == ("transpose_flat", 512, 16 * 399 * 4, 19 * 9)
    # rows too long for a panel of 64 bytes per pixel (71x71: 10082 bytes): the shifted-destination kernel
    assert launch_of(inv(N=32, C=192, H=71, W=71))["kernel"] == "transpose_shifted"
    # a handful of large panels (2 images x 8 panels of 46 KB) would leave most SMs idle: shifted-destination too
    assert launch_of(inv(N=2, C=256, H=27, W=27))["kernel"] == "transpose_shifted"
    assert launch_of(inv(N=20, C=256, H=27, W=27))["kernel"] == "transpose_flat"
    # fewer channels than a panel's 64 bytes, or a channel count that is no multiple of 16 bytes
    assert launch_of(inv(N=2, C=24, H=5, W=13))["kernel"] == "transpose_shifted"
    L = launch_of(inv(N=2, C=68, H=14, W=14))
    assert (L["kernel"], L["access"]) == ("transpose", 8)
    # the other direction (source rows misaligned, destination rows aligned): panels that are contiguous in the
    # source where the rows are short enough and there are enough panels, else the realigning kernel
    fwd = W.c2_nchw_to_nhwc
    L = launch_of(fwd(N=64, C=288, H=35, W=35))
    assert (L["kernel"], L["threads"], L["smem_bytes"], L["n_blocks"]) == ("transpose_flat_source", 512, 78400, 64 * 9)
    L = launch_of(fwd(N=64, C=1024, H=14, W=14))
    assert (L["kernel"], L["threads"], L["smem_bytes"]) == ("transpose_flat_source", 256, 12544)
    assert launch_of(fwd(N=4, C=256, H=27, W=27))["kernel"] == "transpose_realign"
    assert launch_of(fwd(N=32, C=192, H=71, W=71))["kernel"] == "transpose_realign"
    # operands of one concat with enough channels for a panel (40) and with too few (8, 24, 16): all of them on the
    # tiled kernel, so that the transposes stay one launch (plus the launch of the padding borders)
    mixed = B.compose_chain(W.reduced_configs()["c4_odd"]).plan(device=-1).launches()
    assert [l["kernel"] for l in mixed] == ["transpose_realign", "strip"]
    # other families
    assert launch_of(W.full_configs()["c5"])["kernel"] == "strip"
    assert launch_of(W.full_configs()["c3"])["kernel"] in ("affine", "strip")


def test_launch_info_arguments():
    import ctypes

    plan = B.compose_chain(W.full_configs()["c4"]).plan(device=-1)
    (L,) = plan.launches()
    assert L["n_descriptors"] == plan.stats()["n_descriptors"] == 9 and L["stage"] == 0 and L["wide_offsets"] == 0
    info = B._LaunchInfo()
    lib = B._lib
    assert lib.amap_plan_launch_info(plan._h, 1, ctypes.byref(info)) == -1   # one launch only: AMAP_EINVAL
    assert lib.amap_plan_launch_info(plan._h, -1, ctypes.byref(info)) == -1
    assert lib.amap_plan_launch_info(plan._h, 0, None) == -1
    assert lib.amap_plan_launch_info(None, 0, ctypes.byref(info)) == -1


def test_remainders_of_at_most_half_a_tile_become_pieces_of_their_own():
    """The 16-byte transpose kernel's tile spans 128 bytes of the destination run.  An extent that leaves at most
    64 bytes over is cut: whole tiles, plus the remainder on the 64-byte tile."""
    def descriptors(chain):
        return B.compose_chain(chain).plan(device=-1).stats()["n_descriptors"]

    assert descriptors(W.c2_nchw_to_nhwc(N=2, C=128, H=20, W=26)) == 1  # whole tiles only
    assert descriptors(W.c2_nchw_to_nhwc(N=2, C=96, H=20, W=26)) == 2   # 64 + 32 channels
    assert descriptors(W.c2_nchw_to_nhwc(N=2, C=112, H=20, W=26)) == 1  # 48 left over: more than half a tile
    assert descriptors(W.c2_nchw_to_nhwc(N=2, C=24, H=20, W=26)) == 1   # shorter than half a tile altogether
    assert descriptors(W.c2_nchw_to_nhwc(N=2, C=40, H=12, W=23, dtype="fp32")) == 2  # 32 + 8 four-byte elements
    # configuration 4: operands of 64, 96, 128, 32 channels -> five transpose descriptors and four border fills
    assert descriptors(W.full_configs()["c4"]) == 9


def test_unfused_chain_has_one_stage_per_operator_and_moves_more_bytes():
    c3 = W.full_configs()["c3"]
    fused = B.compose_chain(c3).plan(device=-1).stats()
    unfused = B.compose_chain(c3, B.COMPOSE_NO_FUSE).plan(device=-1).stats()
    assert fused["n_stages"] == 1 and unfused["n_stages"] == 7
    assert fused["bytes_read"] + fused["bytes_written"] == 805306368
    assert unfused["bytes_read"] + unfused["bytes_written"] == 3758096384


def test_dry_plan_cannot_execute():
    plan = B.compose_chain(W.c1_small_chain()).plan(device=-1)
    with pytest.raises(B.AmapError) as e:
        plan.execute_ptrs([0x1000], 0x2000, 0)
    assert e.value.code == -1


def test_bad_plan_options():
    m = B.compose_chain(W.c1_small_chain())
    for kw in ({"pointer_align": 3}, {"pointer_align": 2}, {"flags": 64}, {"force_kernel": 9}, {"device": -2}):
        with pytest.raises(B.AmapError) as e:
            m.plan(**{"device": -1, **kw})
        assert e.value.code == -1, kw


def test_execute_entry_points_refuse_bad_buffers_before_any_cuda_call():
    """amap_execute_static shares amap_execute's argument checks: they come before the first CUDA call, so a dry
    plan and made-up addresses show them without a GPU."""
    chain = W.reduced_configs()["c2_fwd_rag"]
    m = B.compose_chain(chain)
    dry = m.plan(device=-1)
    nbytes = m.out_numel * 2
    src = 0x7F0000000000
    codes = {}
    for name, (s, d) in {
        "overlap_equal": (src, src),
        "overlap_partial": (src, src + 64),              # the output starts inside the input
        "overlap_from_below": (src, src - nbytes + 32),  # the output's last bytes reach into the input
        "misaligned_src": (src + 2, src + 4 * nbytes),
        "misaligned_dst": (src, src + 4 * nbytes + 8),
        "null_dst": (src, 0),
    }.items():
        with pytest.raises(B.AmapError) as e:
            dry.execute_static_ptrs([s], d, 0)
        codes[name] = e.value.code
    assert codes == {"overlap_equal": -1, "overlap_partial": -1, "overlap_from_below": -1, "misaligned_src": -7,
                     "misaligned_dst": -7, "null_dst": -1}
    # amap_execute refuses a dry plan outright
    with pytest.raises(B.AmapError) as e:
        dry.execute_ptrs([src], src + 4 * nbytes, 0)
    assert e.value.code == -1


def test_static_entry_point_refuses_temporaries_and_oversized_plans():
    awkward = W.Chain(
        name="awkward", dtype="bf16", inputs=[[40, 24]],
        ops=[
            {"kind": "transpose", "src": 0, "perm": [1, 0]},
            {"kind": "reshape", "src": 1, "shape": [64, 15]},
            {"kind": "transpose", "src": 2, "perm": [1, 0]},
        ],
        values="normal",
    )
    m = B.compose_chain(awkward, B.COMPOSE_NO_FUSE)
    dry = m.plan(device=-1)
    assert dry.stats()["n_stages"] > 1
    with pytest.raises(B.AmapError) as e:
        dry.execute_static_ptrs([0x7F0000000000], 0x7F0000100000, 0)
    assert e.value.code == -9  # temporaries need device memory
    b = B.Builder(2)
    ids = [b.input([4, 8]) for _ in range(22)]
    big = b.compose(b.concat([b.pad(t, [1, 1], [1, 1]) for t in ids], 0)).plan(device=-1)
    assert big.stats()["n_descriptors"] > 64
    with pytest.raises(B.AmapError) as e:
        big.execute_static_ptrs([0x7F0000000000 + 4096 * k for k in range(22)], 0x7F0000100000, 0)
    assert e.value.code == -11
