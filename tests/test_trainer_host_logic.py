"""Host-side logic of the trainer that needs no GPU: the choice of row slices for the dW products."""
import pytest

torch = pytest.importorskip("torch")
from paper_2609_09821_b200 import trainer as T  # noqa: E402


def _bare(np_, kp, max_split=64):
    t = object.__new__(T.MlpTrainer)
    t.max_split, t.Np, t.Kp = max_split, list(np_), list(kp)
    return t


@pytest.mark.parametrize("M", [64, 128, 192, 256, 4096, 32768, 65536, 98304, 262144])
def test_slices_divide_the_rows_into_whole_128_row_blocks(M):
    t = _bare([1024, 1024, 512, 128], [640, 1024, 1024, 512])
    for l in range(4):
        S = t._dw_slices(l, M)
        assert S >= 1 and S & (S - 1) == 0 and S <= t.max_split
        assert S == 1 or M % (128 * S) == 0              # every slice is a whole number of 128-row blocks
        assert S <= t._dw_slices(l, max(M, 1 << 20), any_rows=True)   # the bound the partial buffer is sized by


def test_few_output_tiles_get_many_slices_and_many_tiles_get_few():
    t = _bare([1024, 128], [1024, 512])
    big, small = t._dw_slices(0, 262144), t._dw_slices(1, 262144)
    assert small >= big and small >= 32                  # 2 output tiles need the rows cut up to fill 148 SMs
    assert t._dw_slices(0, 4096) <= 8                    # few rows: the slice-sum pass would cost more than it saves
    assert _bare([1024], [1024], max_split=4)._dw_slices(0, 262144) <= 4
