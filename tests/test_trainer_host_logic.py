"""Host-side logic of the trainer that needs no GPU: the choice of row slices for the dW products
(im_trainer_dw_slices, a pure host function of the C library)."""
import pytest

from paper_2609_09821_b200 import trainer as T


@pytest.mark.parametrize("M", [64, 128, 192, 256, 4096, 32768, 65536, 98304, 262144])
def test_slices_divide_the_rows_into_whole_128_row_blocks(M):
    for Np, Kp in zip([1024, 1024, 512, 128], [640, 1024, 1024, 512]):
        S = T.dw_slices(Np, Kp, M)
        assert S >= 1 and S & (S - 1) == 0 and S <= 64
        assert S == 1 or M % (128 * S) == 0              # every slice is a whole number of 128-row blocks
        assert S <= T.dw_slices(Np, Kp, max(M, 1 << 20), any_rows=True)   # the bound the partial buffer is sized by


def test_few_output_tiles_get_many_slices_and_many_tiles_get_few():
    big, small = T.dw_slices(1024, 1024, 262144), T.dw_slices(128, 512, 262144)
    assert small >= big and small >= 32                  # 2 output tiles need the rows cut up to fill 148 SMs
    assert T.dw_slices(1024, 1024, 4096) <= 8            # few rows: the slice-sum pass would cost more than it saves
    assert T.dw_slices(1024, 1024, 262144, max_split=4) <= 4
