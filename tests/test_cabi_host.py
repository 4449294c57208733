"""CPU-only checks of the C-ABI library: it loads, exports what the header declares, and its host
logic (launch planning, argument validation that needs no device) behaves."""
import ctypes
import os
import re

import pytest

from paper_2308_10037_b200 import api

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2308_10037_b200 import build
    build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "lrgd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lr_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    L = api.lib()
    names = _declared()
    assert "lr_loss_grad" in names and "lr_fit" in names and "lr_predict" in names
    for name in names:
        assert hasattr(L, name), name
    assert sorted(api.EXPORTS) == names


def test_status_strings():
    assert api.status_string(0) == "ok"
    for code in range(-7, 0):
        assert api.status_string(code) not in ("ok", "unknown status")
    assert api.status_string(-99) == "unknown status"


def test_null_context_is_rejected_before_any_cuda_call():
    L = api.lib()
    one = ctypes.c_void_p(16)
    assert L.lr_loss_grad(None, one, one, 4, 4, one, one, one, one, one, None) == api.LR_ERR_NULL
    assert L.lr_fit(None, one, one, 4, 4, 0.1, 1, one, one, None, None) == api.LR_ERR_NULL
    assert L.lr_predict(None, one, 4, 4, one, one, 0.5, one, None) == api.LR_ERR_NULL
    assert L.lr_create(None, 0, 4) == api.LR_ERR_NULL
    h = ctypes.c_void_p()
    assert L.lr_create(ctypes.byref(h), 0, 0) == api.LR_ERR_SHAPE
    assert L.lr_destroy(None) == api.LR_OK


@pytest.mark.parametrize("m,n,lpr,nv,nw", [(10_000, 32, 8, 1, 16), (16_000_000, 64, 16, 1, 16), (1_000_000, 100, 32, 1, 8),
                                            (4_000_000, 256, 32, 2, 16), (11_000_000, 28, 8, 1, 16), (5000, 512, 32, 4, 8),
                                            (70_000, 128, 32, 1, 8), (9_000, 68, 32, 1, 8)])
def test_plan_staged_shapes(m, n, lpr, nv, nw):
    p = api.plan_query(m, n)
    assert p["variant"] == 0 and p["lanes_per_row"] == lpr and p["vec_per_lane"] == nv
    assert p["threads"] == 32 * nw and 1 <= p["grid"] <= 148
    assert p["tile_rows"] == p["rows_per_batch"]              # one stage holds one register batch
    assert 1 <= p["stages"] <= 4
    assert p["smem_bytes"] <= 227 * 1024
    stage = -(-p["tile_rows"] * n * 4 // 128) * 128
    assert 1024 + nw * p["stages"] * stage <= p["smem_bytes"]
    # the warps of a CTA take one batch each per round; the grid never exceeds the rounds available
    batches = -(-m // p["rows_per_batch"])
    # (a problem that fits the shared memory of one thread-block cluster is planned on that cluster's CTAs)
    assert p["grid"] == (api.cluster_ctas(m, n) or min(-(-batches // nw), 148))
    if nw == 8 and nv == 1:
        assert p["rows_per_batch"] == 16                      # 68..128 fp32 columns: sixteen rows per batch, eight warps


def test_plan_for_unaligned_or_odd_shapes():
    # rows of any length in a matrix aligned to its element size: per-warp stages up to 512 columns (variant 3), CTA-wide
    # stages of whole rows up to 16384 (variant 4); only wider rows run unstaged (variant 2)
    assert api.plan_query(1000, 1027)["variant"] == 4        # n not a multiple of 4 and wider than 1024
    assert api.plan_query(1000, 1028, x_aligned16=False)["variant"] == 4   # the row-split kernel needs a 16-byte aligned matrix
    assert api.plan_query(1000, 515)["variant"] == 4 and api.plan_query(1000, 516, x_aligned16=False)["variant"] == 4
    assert api.plan_query(1000, 511)["variant"] == 3 and api.plan_query(1000, 512, x_aligned16=False)["variant"] == 3
    assert api.plan_query(1000, 32, x_aligned16=False)["variant"] == 3     # narrow rows: element-wise staged kernel
    assert api.plan_query(1000, 30, x_aligned16=False)["variant"] == 3
    assert api.plan_query(1000, 32, x_aligned16=False, bf16=True)["variant"] == 3
    assert api.plan_query(1000, 8191)["variant"] == 4 and api.plan_query(1000, 8192, x_aligned16=False)["variant"] == 4
    # beyond the row-split kernel's 8192 columns every row, aligned or not, takes the CTA-wide stages: one row per batch
    for n, nv in ((8193, 24), (8196, 24), (12288, 24), (12289, 32), (16384, 32)):
        for bf16 in (False, True):
            q = api.plan_query(1000, n, bf16=bf16)
            assert (q["variant"], q["vec_per_lane"], q["rows_per_batch"], q["threads"]) == (4, nv, 1, 512)
            assert q["stages"] >= (3 if not bf16 else 4)
    assert api.plan_query(1000, 16385)["variant"] == 2        # wider than any staged kernel
    assert api.plan_query(1000, 16392, bf16=True)["variant"] == 2
    assert api.plan_query(1000, 30, bf16=True)["variant"] == 3   # element-wise staged kernel, bfloat16 too
    assert api.plan_query(1000, 1036, bf16=True)["variant"] == 4 # 1036 % 8 != 0 and wider than 1024
    g = api.plan_query(100, 16389)
    assert g["variant"] == 2 and g["tile_rows"] == 8 and g["grid"] == 13 and g["threads"] == 256   # few rows: 8-row chunks
    g = api.plan_query(200_000, 16389)
    assert g["tile_rows"] == 64 and g["grid"] == 148 * 8                 # enough rows for 64-row chunks on every SM
    w = api.plan_query(100_000, 1027)
    assert w["vec_per_lane"] == 3 and w["rows_per_batch"] == 16 and w["stages"] == 3 and w["threads"] == 512
    assert api.plan_query(100_000, 8191)["rows_per_batch"] == 2
    n513 = api.plan_query(100_000, 513)
    assert n513["rows_per_batch"] == 16 and n513["threads"] == 256 and n513["vec_per_lane"] == 3


@pytest.mark.parametrize("n,lpr,nv,rb", [(1, 2, 1, 2), (3, 4, 1, 4), (7, 8, 1, 8), (13, 16, 1, 16), (30, 32, 1, 32), (33, 32, 2, 16), (101, 32, 4, 8),
                                         (255, 32, 8, 4), (258, 32, 16, 2), (511, 32, 16, 2)])
def test_plan_rows_of_any_length(n, lpr, nv, rb):
    # fp32 rows whose length is not a multiple of four still take a staged kernel: a lane owns single elements
    p = api.plan_query(200_003, n)
    assert p["variant"] == 3 and p["lanes_per_row"] == lpr and p["vec_per_lane"] == nv
    assert p["rows_per_batch"] == rb * (32 // lpr)
    assert nv * lpr >= n and p["smem_bytes"] <= 227 * 1024
    stage = -(-(p["tile_rows"] * n * 4 + 16) // 128) * 128      # a batch may start up to 12 bytes into its stage
    assert 1024 + 16 * p["stages"] * stage <= p["smem_bytes"]


def test_plan_rows_of_516_to_1024_columns_use_eight_warps():
    for m, n in [(5000, 516), (5000, 1024), (200_000, 1000)]:
        p = api.plan_query(m, n)
        assert p["variant"] == 0 and p["threads"] == 256 and p["rows_per_batch"] == 2
        assert p["vec_per_lane"] == -(-(n // 4) // 32)                # 129..256 groups: five to eight per lane, no more than needed
        stage = -(-2 * n * 4 // 128) * 128
        assert 1024 + 8 * p["stages"] * stage <= p["smem_bytes"] <= 227 * 1024
        assert p["smem_bytes"] >= 1024 + 8 * n * 8 + 2 * 8 * 8         # room for the end-of-kernel combine of eight warps
        assert p["grid"] == min(-(-(-(-m // 2)) // 8), 148)
    pb = api.plan_query(5000, 1024, bf16=True)                        # bfloat16: 65..128 groups per row, eight warps too
    assert pb["variant"] == 0 and pb["threads"] == 256 and pb["vec_per_lane"] == 4 and pb["rows_per_batch"] == 2
    assert api.plan_query(5000, 1032, bf16=True)["variant"] == 1     # wider bfloat16 rows stay on the split kernel


@pytest.mark.parametrize("m,n,nv,rb", [(100_000, 4096, 2, 4), (5000, 1028, 1, 16), (5000, 1540, 1, 8), (5000, 2052, 2, 8), (5000, 3200, 2, 4), (5000, 6148, 4, 2), (5000, 8192, 4, 2)])
def test_plan_wide_rows_are_split_across_warps(m, n, nv, rb):
    p = api.plan_query(m, n)
    assert p["variant"] == 1 and p["vec_per_lane"] == nv and p["rows_per_batch"] == rb
    assert p["threads"] == 512 and p["grid"] == min(-(-m // rb), 148)
    cw = -(-(n // 4) // 16)
    stage = -(-rb * cw * 16 // 128) * 128
    assert 1 <= p["stages"] <= 4 and p["smem_bytes"] == 4096 + 16 * p["stages"] * stage <= 227 * 1024


def test_plan_rejects_bad_shapes():
    for m, n in [(0, 4), (4, 0), (-1, 4), (1 << 41, 4)]:
        with pytest.raises(api.LrError) as e:
            api.plan_query(m, n)
        assert e.value.code == api.LR_ERR_SHAPE


def test_pipeline_depth_follows_the_shared_memory_budget():
    assert api.plan_query(4_000_000, 256)["stages"] == 3        # 4 KB batches: three per warp fit
    assert api.plan_query(16_000_000, 64)["stages"] == 3
    assert api.plan_query(1_000_000, 100)["stages"] == 4        # 3.2 KB batches
    assert api.plan_query(100, 32)["stages"] == 1               # one batch per warp at most


@pytest.mark.parametrize("m,n,bf16,aligned,want", [
    (10_000, 32, False, True, 16),      # two batches of 32 rows for most warps of 16 CTAs
    (4_100, 32, False, True, 8),        # 9 CTA-loads of batches: not enough for sixteen CTAs, enough for eight
    (3_000, 32, False, True, 0),        # 6 CTA-loads: too few even for a cluster of eight
    (24_000, 32, False, True, 16),      # three stages per warp
    (30_001, 32, False, True, 0),       # four stages of 4 KB per warp do not fit beside the received rows
    (30_001, 32, True, True, 16),       # ... with bfloat16 rows they do
    (60_000, 32, False, True, 0),       # more rows than a cluster's shared memory holds
    (1_500, 256, False, True, 16),
    (3_000, 256, False, True, 0),
    (3_000, 100, False, True, 16),      # an eight-warp shape
    (10_000, 32, False, False, 0),      # rows that are not 16-byte groups
    (10_000, 30, False, True, 0),
    (2_000, 1028, False, True, 0),      # wide rows have no persistent form
])
def test_cluster_plan(m, n, bf16, aligned, want):
    C = api.cluster_ctas(m, n, x_aligned16=aligned, bf16=bf16)
    assert C == want
    if C:
        # every entry point plans the problem on C CTAs, all of them busy, all batches of a warp resident at once
        p = api.plan_query(m, n, bf16=bf16)
        assert p["variant"] == 0 and p["grid"] == C
        assert api.cluster_ctas(m, n, sm_count=C, bf16=bf16) == C and api.cluster_ctas(m, n, sm_count=7, bf16=bf16) == 0
        assert api.plan_query(m, n, sm_count=7, bf16=bf16)["grid"] == 7
        warps = p["threads"] // 32
        batches = -(-m // p["rows_per_batch"])
        per_warp = -(-(-(-batches // warps)) // C)
        assert per_warp <= 4
        stage = -(-(p["rows_per_batch"] * n * (2 if bf16 else 4)) // 128) * 128
        assert warps * per_warp * stage + 2 * C * (n + 2) * 8 < 227 * 1024


def test_header_is_plain_c_and_the_example_links():
    # include/lrgd.h must be usable from C (no C++ in the boundary); the example program must compile and link against the
    # built library (it is only run where a GPU exists)
    import shutil
    import subprocess
    import tempfile
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no gcc")
    inc = os.path.join(ROOT, "include")
    pkg = os.path.join(ROOT, "paper_2308_10037_b200")
    with tempfile.TemporaryDirectory() as tmp:
        probe = os.path.join(tmp, "probe.c")
        with open(probe, "w") as f:
            f.write('#include "lrgd.h"\nint main(void) { lr_plan p; return lr_plan_query(10, 4, 1, 148, &p) == LR_OK ? 0 : 1; }\n')
        subprocess.check_call([gcc, "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", inc, probe, "-L", pkg, "-llrgd",
                               f"-Wl,-rpath,{pkg}", "-o", os.path.join(tmp, "probe")])
        subprocess.check_call([os.path.join(tmp, "probe")])          # pure host entry point: runs without a GPU
        subprocess.check_call([gcc, "-std=c99", "-Wall", "-Werror", "-O1", "-I", inc, os.path.join(pkg, "examples", "fit_host.c"),
                               "-L", pkg, "-llrgd", f"-Wl,-rpath,{pkg}", "-lm", "-o", os.path.join(tmp, "fit_host")])


def test_any_length_copies_stay_inside_the_matrix():
    """The staged kernel for rows of any length copies, per batch, the 16-byte-aligned span that starts at or just before
    the batch (at the first boundary inside it for the first batch of a matrix that is not 16-byte aligned) and ends at or
    before its last byte, and moves the few words left over with plain loads.  This replays that arithmetic for every
    batch of many shapes and base alignments: aligned bulk copies, nothing read outside the matrix, every byte of the
    matrix covered exactly once, nothing written outside the stage."""
    import random
    rnd = random.Random(1)
    shapes = [(2758, 449), (1, 1), (7, 3), (300, 1), (640, 30), (1025, 101), (526, 255), (999, 511), (5, 510), (3, 258),
              (17, 257), (2, 449), (1, 511), (40, 8193), (33, 12291), (19, 16383), (7, 16384)]
    shapes += [(rnd.randint(1, 3000), rnd.choice([n for n in range(1, 513) if n % 4])) for _ in range(200)]
    shapes += [(3, 513), (1, 1023), (77, 1021), (500, 777), (2, 1022), (9, 8191), (33, 4099), (5, 2049), (64, 1025)]
    shapes += [(rnd.randint(1, 400), rnd.choice([n for n in range(513, 8192) if n % 4])) for _ in range(60)]
    cases = [(m, n, 0, 4) for m, n in shapes]
    extra = shapes[:60] + [(1, 1), (2, 2), (3, 1), (40, 32), (999, 256), (77, 512)]
    cases += [(m, n, base, 4) for (m, n) in extra for base in (4, 8, 12)]
    # bfloat16 (2-byte elements): lengths that are not a multiple of eight, and bases on every even offset
    cases += [(m, n, 0, 2) for (m, n) in shapes[:80] if n % 8] + [(m, n, base, 2) for (m, n) in extra[:40] for base in (2, 6, 10, 14)]
    for m, n, base, eb in cases:
        p = api.plan_query(m, n, x_aligned16=(base == 0), bf16=(eb == 2))
        assert p["variant"] == (3 if n <= 512 else 4)             # per-warp stages up to 512 columns, CTA-wide stages beyond
        rpb, row_bytes = p["rows_per_batch"], eb * n
        lo_x, hi_x = 4096 + base, 4096 + base + eb * m * n         # the matrix occupies the addresses [lo_x, hi_x)
        stage = -(-(rpb * row_bytes + 16) // 128) * 128
        if p["variant"] == 3:
            assert 1024 + (p["threads"] // 32) * p["stages"] * stage <= p["smem_bytes"]
        else:
            assert 4096 + p["stages"] * stage == p["smem_bytes"] <= 227 * 1024
        seen = 0
        for g in range(-(-m // rpb)):
            r0 = g * rpb
            xbytes = min(rpb, m - r0) * row_bytes
            src = lo_x + r0 * row_bytes
            off = src & 15
            span = off + xbytes
            lo = 16 if (r0 == 0 and off != 0) else 0
            bulk = ((span - lo) & ~15) if span > lo else 0
            assert span <= stage
            if bulk:
                assert (src - off + lo) % 16 == 0 and lo_x <= src - off + lo and src - off + lo + bulk <= hi_x
            head = list(range(off, min(lo, span), eb))
            tail = list(range(lo + bulk, span, eb))
            assert len(head) <= 16 // eb - 1 and len(tail) <= 16 // eb - 1
            assert all(lo_x <= src - off + o and src - off + o + eb <= hi_x for o in head + tail)
            # every byte of the batch is written exactly once: head, bulk and tail tile [off, span) of the stage
            written = sorted(head + tail + list(range(lo, lo + bulk, eb)))
            assert [o for o in written if o >= off] == list(range(off, span, eb))
            seen += xbytes
        assert seen == eb * m * n


def test_every_row_length_gets_a_launchable_plan():
    """Sweeps n = 1 .. 16500 for both storage types and both alignments: the plan always names a kernel shape that exists,
    fits the shared memory of a CTA, keeps at least one stage, and (staged kernels) sizes its stages as the kernels do."""
    for bf16 in (False, True):
        eb, epg = (2, 8) if bf16 else (4, 4)
        for aligned in (True, False):
            for n in list(range(1, 1100)) + list(range(1100, 8301, 4)) + list(range(8301, 16500, 52)) + [4097, 8191, 8193, 12288, 12289, 16383, 16384, 16385, 16388]:
                p = api.plan_query(70_001, n, x_aligned16=aligned, bf16=bf16)
                v = p["variant"]
                assert p["smem_bytes"] <= 227 * 1024 and p["grid"] >= 1 and p["threads"] in (256, 512)
                if v in (0, 3):
                    nw = p["threads"] // 32
                    assert nw in (8, 16) and 1 <= p["stages"] <= 4
                    lanes = p["lanes_per_row"]
                    groups = n if v == 3 else n // epg
                    assert lanes in (2, 4, 8, 16, 32)
                    assert p["vec_per_lane"] * lanes >= groups and (lanes >= 8 or groups <= lanes)
                    assert p["rows_per_batch"] % (32 // lanes) == 0
                    stage = -(-(p["rows_per_batch"] * n * eb + (16 if v == 3 else 0)) // 128) * 128
                    assert 1024 + nw * p["stages"] * stage <= p["smem_bytes"]
                    assert p["smem_bytes"] >= 1024 + nw * n * 8 + 2 * nw * 8          # the end-of-kernel combine
                    if v == 0:
                        assert aligned and n % epg == 0
                    else:
                        assert n <= 512
                elif v == 4:
                    # wide rows of any length: CTA-wide stages of whole rows; eight warps up to 1024 elements, sixteen beyond
                    nw = p["threads"] // 32
                    assert 512 < n <= 16384 and nw == (8 if n <= 1024 else 16)
                    # rows of any length or alignment, and the aligned fp32 rows of 4100..6144 columns the row-split kernel is weak on
                    assert not (aligned and n % epg == 0) or (not bf16 and 4096 < n <= 6144) or n > 8192
                    cw = -(-n // nw)
                    assert p["vec_per_lane"] in (2, 3, 4, 6, 8, 12, 16, 24, 32) and p["vec_per_lane"] * 32 >= cw
                    assert p["vec_per_lane"] * p["rows_per_batch"] in (24, 32, 48, 64) and p["rows_per_batch"] in (1, 2, 4, 8, 16)
                    assert (p["rows_per_batch"] == 1) == (n > 8192)
                    assert 2 * nw * p["rows_per_batch"] * 4 <= 4096 - 1024                   # the logit exchange fits the header
                    stage = -(-(p["rows_per_batch"] * n * eb + 16) // 128) * 128
                    assert 1 <= p["stages"] <= 4 and p["smem_bytes"] == 4096 + p["stages"] * stage
                elif v == 1:
                    nw = p["threads"] // 32
                    assert aligned and n % epg == 0 and nw == (8 if bf16 else 16)
                    assert bf16 or not (4096 < n <= 6144)
                    cw = -(-(n // epg) // nw)
                    assert p["vec_per_lane"] * 32 >= cw and p["vec_per_lane"] in (1, 2, 4)
                    assert cw * (2 if cw > 64 else 4) <= 256                                   # tensor-map box limit (64-bit words beyond 64 groups)
                    assert 2 * nw * p["rows_per_batch"] * 4 <= 4096 - 1024                   # the logit exchange fits the header
                    stage = -(-p["rows_per_batch"] * cw * 16 // 128) * 128
                    assert 1 <= p["stages"] <= 4 and p["smem_bytes"] == 4096 + nw * p["stages"] * stage
                else:
                    assert v == 2 and p["threads"] == 256 and n > 16384
