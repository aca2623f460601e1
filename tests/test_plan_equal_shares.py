"""Host logic of the equal-share launch (no GPU): the cut of the tile-major (tile, group) list into one
contiguous range per CTA that rosaq_linear uses when a launch has at least one column tile per SM."""
import pytest

from paper_2506_13472_b200 import binding as rb

FP16_COST, QUANT_COST = 3, 2          # an fp16 group counts 1.5 quantized ones


def cost(lo, hi, groups, g_fp16):
    return sum(FP16_COST if (u % groups) < g_fp16 else QUANT_COST for u in range(lo, hi))


@pytest.mark.parametrize("n_tiles,groups,g_fp16,n_ctas", [
    (172, 32, 1, 296),        # gate + up of a 7B layer in one launch
    (96, 32, 1, 296),         # q + k + v
    (86, 86, 86, 296),        # a dense 11008 x 11008 rotation operand (every group fp16)
    (216, 40, 1, 296),        # gate + up at 13B size
    (150, 8, 1, 296),         # the small case of the GPU tests
    (296, 5, 0, 296),         # one tile per CTA exactly
    (7, 64, 2, 20),
])
def test_cut_covers_the_list_in_equal_contiguous_shares(n_tiles, groups, g_fp16, n_ctas):
    b = rb.plan_equal_shares(n_tiles, groups, g_fp16, n_ctas)
    assert len(b) == n_ctas + 1 and b[0] == 0 and b[-1] == n_tiles * groups
    assert all(b[i] < b[i + 1] for i in range(n_ctas))                     # no empty range
    assert all((b[i + 1] - 1) // groups - b[i] // groups <= 1 for i in range(n_ctas))   # two tiles at most
    total = cost(0, n_tiles * groups, groups, g_fp16)
    shares = [cost(b[i], b[i + 1], groups, g_fp16) for i in range(n_ctas)]
    assert sum(shares) == total
    # every cut is the exact position rounded down to a group boundary: a share is off by less than a group
    assert max(shares) - total / n_ctas < FP16_COST + 1e-9
    assert total / n_ctas - min(shares) < FP16_COST + 1e-9


@pytest.mark.parametrize("args,status", [
    ((10, 2, 1, 296), rb.ROSAQ_ERR_UNSUPPORTED_SHAPE),     # fewer groups than CTAs: some range is empty
    ((300, 4, 0, 100), rb.ROSAQ_ERR_UNSUPPORTED_SHAPE),    # three tiles per CTA
    ((0, 4, 0, 8), rb.ROSAQ_ERR_INVALID_ARG),
    ((4, 4, 5, 8), rb.ROSAQ_ERR_INVALID_ARG),
    ((4, 4, 1, 0), rb.ROSAQ_ERR_INVALID_ARG),
])
def test_unusable_cuts_are_status_codes(args, status):
    with pytest.raises(rb.RosaqError) as e:
        rb.plan_equal_shares(*args)
    assert e.value.status == status
