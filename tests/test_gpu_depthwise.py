"""Depthwise 3x3 layers at sizes that select the row-walking kernel (one thread walks up to 16
output rows of its columns), against the oracle through the C ABI.  The small networks of the
other forward tests stay on the one-row-per-thread kernel, so these cases are the parity cover
of the row-walking one: stride 1 and 2, a shortcut into a depthwise layer, row blocks of equal
and of unequal height, a single block per image, an odd width, and a channel count whose last
octet is partly padding."""
import numpy as np
import pytest

from aiq_workloads import depthwise_stack, gen_model, gen_images
from oracle import aiq_oracle as O
from gpu_util import binding, to_dev, assert_logits_close, compute_path

pytestmark = pytest.mark.gpu


# (image size, channels, batch): output heights of the two depthwise layers = size / 2; the batch
# is what it takes to give each of 148 SMs a block of threads
CASES = [
    (64, 192, 52),    # 32 rows: two blocks of 16
    (56, 192, 60),    # 28 rows: two blocks of 14
    (42, 188, 76),    # 21 x 21 (odd width): blocks of 11 and 10 rows; 188 channels (4 padding channels)
    (28, 192, 228),   # 14 rows: one block
]


SCHEMES = ([8, 8, 8, 8, 8], [8, 4, 8, 32, 8])
_REFS = {}


def _case(hw, channels, batch):
    """Architecture, parameters, images and the oracle's logits per scheme (computed once per case)."""
    key = (hw, channels, batch)
    if key not in _REFS:
        arch = depthwise_stack(hw, channels)
        params = gen_model(arch, 9000 + hw)
        bank = O.build_weight_bank(O.fold_model(arch, params), (4, 8, 32))
        x = gen_images(batch, 3, hw, hw, 9100 + hw)
        refs = [O.forward_scheme(arch, bank, np.array(sc, np.uint8), x) for sc in SCHEMES]
        _REFS[key] = (arch, params, x, refs)
    return _REFS[key]


@pytest.mark.parametrize("path", ["fp32", "tensor"])
@pytest.mark.parametrize("hw,channels,batch", CASES)
def test_depthwise_row_walking_kernel(hw, channels, batch, path):
    aiq = binding()
    arch, params, x, refs = _case(hw, channels, batch)
    with compute_path(path):
        model = aiq.Model(arch, params)
    xd = to_dev(x)
    for sc, ref in zip(SCHEMES, refs):
        got = model.aiq_forward(np.array(sc, np.uint8), xd).cpu().numpy()
        assert_logits_close(got, ref, f"depthwise stack {hw} {path} {sc}")
    model.close()
