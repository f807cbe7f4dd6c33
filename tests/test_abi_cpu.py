"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol the header declares, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_1810_05486_b200 import build
    build.build()
    from paper_1810_05486_b200 import binding
    return binding


def header_functions():
    text = open(os.path.join(ROOT, "include", "kahan_sgd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kahan_sgd_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol(B):
    names = header_functions()
    assert len(names) >= 10
    for name in names:
        assert hasattr(B.lib, name), name
    assert sorted(B.EXPORTS) == names


def test_desc_struct_layout_matches_header(B):
    assert ctypes.sizeof(B.ksgd_tensor_desc) == 48
    assert B.ksgd_tensor_desc.numel.offset == 16
    assert B.ksgd_tensor_desc.exp_theta_next.offset == 40


def good(**over):
    d = dict(theta=0x10000, comp=0x20000, numel=1000, theta_bits=8, comp_bits=8, overlap_k=0,
             exp_theta=-11)
    d.update(over)
    return d


@pytest.mark.parametrize("desc,code", [
    (good(theta_bits=4), "KSGD_ERR_BITS"),
    (good(comp_bits=12), "KSGD_ERR_BITS"),
    (good(theta=0), "KSGD_ERR_NULL"),
    (good(comp=0), "KSGD_ERR_NULL"),
    (good(comp_bits=0), "KSGD_ERR_NULL"),          # comp given but no compensation asked for
    (good(overlap_k=8), "KSGD_ERR_OVERLAP"),
    (good(overlap_k=-1), "KSGD_ERR_OVERLAP"),
    (good(numel=0), "KSGD_ERR_NUMEL"),
    (good(numel=(1 << 40) + 1), "KSGD_ERR_NUMEL"),  # beyond the index field of a tile table entry
    (good(exp_theta=65), "KSGD_ERR_EXP_RANGE"),
    (good(exp_theta=-65), "KSGD_ERR_EXP_RANGE"),
    (good(exp_theta=0, exp_theta_next=9), "KSGD_ERR_EXP_RANGE"),
    (good(theta=0x10008), "KSGD_ERR_ALIGN"),
    (good(comp=0x20004), "KSGD_ERR_ALIGN"),
])
def test_init_rejects_bad_descriptions_without_cuda(B, desc, code):
    descs = B.make_descs([desc])
    assert B.kahan_sgd_workspace_bytes(descs) == 0
    with pytest.raises(B.KahanSgdError) as ei:
        B.kahan_sgd_init(descs, B.KSGD_EXP_AMAX, 0x100000, 1 << 20)
    assert ei.value.code == getattr(B, code)


def test_init_rejects_bad_workspace_and_mode(B):
    descs = B.make_descs([good()])
    need = B.kahan_sgd_workspace_bytes(descs)
    assert need > 0 and need % 256 == 0
    for args, code in (((B.KSGD_EXP_AMAX, 0, need), B.KSGD_ERR_NULL),
                       ((B.KSGD_EXP_AMAX, 0x100010, need), B.KSGD_ERR_ALIGN),
                       ((B.KSGD_EXP_AMAX, 0x100000, need - 1), B.KSGD_ERR_WORKSPACE),
                       ((7, 0x100000, need), B.KSGD_ERR_MODE)):
        with pytest.raises(B.KahanSgdError) as ei:
            B.kahan_sgd_init(descs, *args)
        assert ei.value.code == code
    assert B.lib.kahan_sgd_init(None, descs, 1, 1, 0x100000, need, None) == B.KSGD_ERR_NULL


def test_workspace_grows_with_the_chunk_table(B):
    small = B.kahan_sgd_workspace_bytes(B.make_descs([good(numel=10)]))
    large = B.kahan_sgd_workspace_bytes(B.make_descs([good(numel=10_000_000)]))
    many = B.kahan_sgd_workspace_bytes(B.make_descs([good(numel=10)] * 500))
    assert small < large and small < many
    # ~8 bytes per 8192-element chunk: a billion parameters need about a megabyte
    big = B.kahan_sgd_workspace_bytes(B.make_descs([good(numel=1_000_000_000, theta_bits=16,
                                                         comp_bits=16)]))
    assert big < 2 << 20


def test_long_lists_of_8bit_theta_get_the_large_tiles(B):
    """The tile tables (8 bytes per tile) show which tile sizes a list got.  First table: 8192
    elements, or 16384 for 8-bit theta once the list still has 1024 tiles with them; 16-bit
    theta always keeps 8192.  A second table, for steps on 8-bit gradients, once the list has
    1024 tiles of twice those sizes (32768 for 8-bit theta with an 8-bit c, 16384 otherwise).
    Every table reserves 1024 entries more than it has whole tiles, for the pieces its last
    round over the blocks is cut into (the size query does not know the device)."""
    reserve = 8 * 1024

    def table_bytes(numel, **kw):        # the first table's reserve cancels in the difference
        return (B.kahan_sgd_workspace_bytes(B.make_descs([good(numel=numel, **kw)])) -
                B.kahan_sgd_workspace_bytes(B.make_descs([good(numel=1, **kw)])))
    short, long_ = 1023 * 16384, 1024 * 16384
    assert abs(table_bytes(short) - 8 * (short // 8192)) <= 512          # small tiles, one table
    assert abs(table_bytes(long_) - 8 * 1024) <= 512                     # large tiles, one table
    longer = 1024 * 32768
    assert abs(table_bytes(longer) - 8 * (2048 + 1024) - reserve) <= 512   # and 1024 tiles of 32768 in the second
    wide = dict(theta_bits=16, comp_bits=16)
    assert abs(table_bytes(short, **wide) - 8 * (short // 8192)) <= 512  # 16-bit theta: small tiles, one table
    assert abs(table_bytes(long_, **wide) - 8 * (long_ // 8192 + 1024) - reserve) <= 512   # second table: 1024 tiles of 16384
    mixed = dict(theta_bits=8, comp_bits=16)                             # 8-bit theta with a 16-bit c: 16384 in both
    assert abs(table_bytes(long_, **mixed) - 8 * (1024 + 1024) - reserve) <= 512
    # a one-element list: the table is the reserve and little else
    assert B.kahan_sgd_workspace_bytes(B.make_descs([good(numel=1)])) < reserve + 4096


def test_null_handles_and_strerror(B):
    assert B.lib.kahan_sgd_step(None, None, None) == B.KSGD_ERR_NULL
    assert B.lib.kahan_sgd_amax(None, *([None] * 7)) == B.KSGD_ERR_NULL
    assert B.lib.kahan_sgd_set_exponents(None, None) == B.KSGD_ERR_NULL
    assert B.lib.kahan_sgd_destroy(None) == B.KSGD_ERR_NULL
    assert B.lib.kahan_sgd_step_host(None, None, None, None, None, None, 0) == B.KSGD_ERR_NULL
    seen = {B.kahan_sgd_strerror(c) for c in range(0, -12, -1)}
    assert len(seen) == 12 and "unknown error code" not in seen
    assert B.kahan_sgd_strerror(-99) == "unknown error code"
    assert B.kahan_sgd_launch_count() == 0          # nothing was launched by these checks


def test_momentum_init_rejects_bad_descriptions_without_cuda(B):
    assert ctypes.sizeof(B.ksgd_momentum_desc) == 24
    ok_m = dict(mom=0x30000, mom_bits=8, exp_mom=-14)
    cases = [((good(), dict(ok_m, mom_bits=4)), B.KSGD_ERR_BITS),
             ((good(comp_bits=0, comp=0), ok_m), B.KSGD_ERR_BITS),      # momentum needs the lazy update
             ((good(), dict(ok_m, mom=0)), B.KSGD_ERR_NULL),
             ((good(), dict(ok_m, mom=0x30004)), B.KSGD_ERR_ALIGN),
             ((good(), dict(ok_m, exp_mom=70)), B.KSGD_ERR_EXP_RANGE),
             ((good(), dict(ok_m, exp_mom=0, exp_mom_next=-9)), B.KSGD_ERR_EXP_RANGE)]
    for (d, m), code in cases:
        descs, mdescs = B.make_descs([d]), B.make_momentum_descs([m])
        assert B.kahan_sgd_momentum_workspace_bytes(descs, mdescs) == 0
        with pytest.raises(B.KahanSgdError) as ei:
            B.kahan_sgd_momentum_init(descs, mdescs, B.KSGD_EXP_AMAX, 0x100000, 1 << 20)
        assert ei.value.code == code
    many = [good()] * 257                 # long lists are allowed (arguments go through the workspace)
    assert B.kahan_sgd_momentum_workspace_bytes(B.make_descs(many), B.make_momentum_descs([ok_m] * 257)) > 0
    assert B.kahan_sgd_momentum_workspace_bytes(B.make_descs([good()]), B.make_momentum_descs([ok_m])) > 0
    assert B.lib.kahan_sgd_momentum_step(None, None, None, None) == B.KSGD_ERR_NULL
    assert B.lib.kahan_sgd_momentum_amax(None, *([None] * 11)) == B.KSGD_ERR_NULL
    assert B.lib.kahan_sgd_momentum_destroy(None) == B.KSGD_ERR_NULL


def test_adam_init_rejects_bad_descriptions_without_cuda(B):
    assert ctypes.sizeof(B.ksgd_adam_desc) == 32 and ctypes.sizeof(B.ksgd_adam_stats) == 15 * 8
    ok_a = dict(mom1=0x30000, mom2=0x40000, exp_m=-20, exp_v=-36)
    cases = [((good(comp_bits=0, comp=0), ok_a), B.KSGD_ERR_BITS),      # ADAM needs the lazy update
             ((good(), dict(ok_a, mom1=0)), B.KSGD_ERR_NULL),
             ((good(), dict(ok_a, mom2=0)), B.KSGD_ERR_NULL),
             ((good(), dict(ok_a, mom2=0x40002)), B.KSGD_ERR_ALIGN),
             ((good(), dict(ok_a, exp_m=-70)), B.KSGD_ERR_EXP_RANGE),
             ((good(), dict(ok_a, exp_v=65)), B.KSGD_ERR_EXP_RANGE),
             ((good(), dict(ok_a, exp_v=0, exp_v_next=9)), B.KSGD_ERR_EXP_RANGE),
             ((good(), dict(ok_a, exp_m=0, exp_m_next=-9)), B.KSGD_ERR_EXP_RANGE)]
    for (d, a), code in cases:
        descs, adescs = B.make_descs([d]), B.make_adam_descs([a])
        assert B.kahan_sgd_adam_workspace_bytes(descs, adescs) == 0
        with pytest.raises(B.KahanSgdError) as ei:
            B.kahan_sgd_adam_init(descs, adescs, B.KSGD_EXP_AMAX, 0x100000, 1 << 20)
        assert ei.value.code == code
    assert B.kahan_sgd_adam_workspace_bytes(B.make_descs([good()] * 257), B.make_adam_descs([ok_a] * 257)) > 0
    descs, adescs = B.make_descs([good()]), B.make_adam_descs([ok_a])
    need = B.kahan_sgd_adam_workspace_bytes(descs, adescs)
    assert need > 0 and need % 256 == 0
    for ws, nb, mode, code in ((0, need, B.KSGD_EXP_AMAX, B.KSGD_ERR_NULL),
                               (0x100010, need, B.KSGD_EXP_AMAX, B.KSGD_ERR_ALIGN),
                               (0x100000, need - 1, B.KSGD_EXP_AMAX, B.KSGD_ERR_WORKSPACE),
                               (0x100000, need, 7, B.KSGD_ERR_MODE)):
        with pytest.raises(B.KahanSgdError) as ei:
            B.kahan_sgd_adam_init(descs, adescs, mode, ws, nb)
        assert ei.value.code == code
    assert B.lib.kahan_sgd_adam_step(None, None, None, 0.9, 0.999, 1e-8) == B.KSGD_ERR_NULL
    assert B.lib.kahan_sgd_adam_amax(None, None) == B.KSGD_ERR_NULL
    assert B.lib.kahan_sgd_adam_destroy(None) == B.KSGD_ERR_NULL
    assert B.lib.kahan_sgd_adam_selfcheck(None, None, None) == B.KSGD_ERR_NULL
    assert B.kahan_sgd_launch_count() == 0


def test_strict_and_fixed_point_gradient_entry_points_reject_bad_arguments_without_cuda(B):
    descs = B.make_descs([good()])
    assert B.kahan_sgd_strict_workspace_bytes(descs, [-18]) > 0
    for d, ec, nxt, code in [(good(comp_bits=0, comp=0), [-18], None, B.KSGD_ERR_BITS),
                             (good(), [-11 - 37], None, B.KSGD_ERR_EXP_RANGE),      # e - ec = 37
                             (good(), [-11 + 9], None, B.KSGD_ERR_EXP_RANGE),       # e - ec = -9
                             (good(), [-18], [-11 - 40], B.KSGD_ERR_EXP_RANGE),
                             # inside both windows, but c's exponent would move by 17 in one step
                             (good(exp_theta=0, exp_theta_next=8), [-20], [-3], B.KSGD_ERR_EXP_RANGE),
                             (good(exp_theta=-40), [-70], None, B.KSGD_ERR_EXP_RANGE)]:
        ds = B.make_descs([d])
        if nxt is None:
            assert B.kahan_sgd_strict_workspace_bytes(ds, ec) == 0
        with pytest.raises(B.KahanSgdError) as ei:
            B.kahan_sgd_strict_init(ds, ec, nxt, B.KSGD_EXP_AMAX, 0x100000, 1 << 20)
        assert ei.value.code == code
    # A state taken from a running handle: c's stored exponent lies in the window of theta's
    # stored exponent only (theta moves 8 up, c's next exponent with it).  The size query
    # must accept it: the exponents of the first step are init's to check.
    resumed = B.make_descs([good(exp_theta=0, exp_theta_next=8)])
    assert B.kahan_sgd_strict_workspace_bytes(resumed, [-36]) > 0
    with pytest.raises(B.KahanSgdError) as ei:       # ... and init refuses it without its next exponent
        B.kahan_sgd_strict_init(resumed, [-36], None, B.KSGD_EXP_AMAX, 0x100000, 1 << 20)
    assert ei.value.code == B.KSGD_ERR_EXP_RANGE
    assert B.lib.kahan_sgd_strict_init(None, descs, None, None, 1, 1, None, 0, None) == B.KSGD_ERR_NULL
    assert B.lib.kahan_sgd_strict_exponents(None, None, None) == B.KSGD_ERR_NULL
    assert B.lib.kahan_sgd_step_qgrad(None, None, 8, None, None) == B.KSGD_ERR_NULL
    assert B.kahan_sgd_launch_count() == 0


def test_classifier_bits_follow_eq_5_and_the_printed_example(B):
    import math
    rows = [ln.split() for ln in open(os.path.join(ROOT, "tests", "golden", "classifier_bitwidth.txt"))
            if ln.strip() and not ln.startswith("#")]
    for classes, alpha, bound, bits in rows:
        classes, alpha, bound, bits = int(classes), float(alpha), float(bound), int(bits)
        assert abs(math.log2(classes - 1) + math.log2(2 / alpha) - bound) < 0.01
        assert B.kahan_sgd_classifier_bits(classes, alpha) == bits
    for classes in (2, 3, 5, 100, 1000, 21841):
        for alpha in (0.5, 0.25, 0.1):
            b = B.kahan_sgd_classifier_bits(classes, alpha)
            real = math.log2(classes - 1) + math.log2(2 / alpha)
            assert b > real and b - 1 <= real + 1e-12        # smallest integer strictly above
    assert B.kahan_sgd_classifier_bits(1, 0.5) == 0 and B.kahan_sgd_classifier_bits(10, 0.0) == 0
    assert B.kahan_sgd_classifier_bits(10, 1.0) == 0


def test_import_export_reject_bad_arguments_without_cuda(B):
    imp, exp = B.lib.kahan_sgd_import, B.lib.kahan_sgd_export
    assert imp(0x1000, 0x2000, 0x3000, 10, 4, 8, 0, 0, None, None, None) == B.KSGD_ERR_BITS
    assert imp(0x1000, 0x2000, 0x3000, 10, 8, 8, 9, 0, None, None, None) == B.KSGD_ERR_OVERLAP
    assert imp(None, 0x2000, 0x3000, 10, 8, 8, 0, 0, None, None, None) == B.KSGD_ERR_NULL
    assert imp(0x1000, 0x2000, None, 10, 8, 8, 0, 0, None, None, None) == B.KSGD_ERR_NULL
    assert imp(0x1000, 0x2000, 0x3000, 0, 8, 8, 0, 0, None, None, None) == B.KSGD_ERR_NUMEL
    assert imp(0x1000, 0x2000, 0x3000, 10, 8, 8, 0, 65, None, None, None) == B.KSGD_ERR_EXP_RANGE
    assert imp(0x1000, 0x2000, 0x3000, 10, 8, 8, 0, B.KSGD_EXP_AUTO, None, None, None) == B.KSGD_ERR_NULL
    assert exp(0x2000, 0x3000, None, 10, 8, 8, 0, 0, None) == B.KSGD_ERR_NULL
    assert exp(0x2000, 0x3000, 0x1000, 10, 8, 8, 0, -70, None) == B.KSGD_ERR_EXP_RANGE
