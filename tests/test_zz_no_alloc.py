"""The scratch-free confidence entry point against the ordinary one (collected last on purpose).

`polestar_k_confidence_noalloc` serves callers that cannot allocate or pass device scratch; it must
give exactly what `polestar_k_confidence` gives, call after call, while reusing one built-in array."""
import numpy as np
import pytest
import torch

from paper_2607_14107_b200 import binding as Bd
from paper_2607_14107_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _run_pair(rows, V, seed):
    logits = I.normal_tensor(I.tensor_key(seed, -1, 7), (rows, V), 3.0).cuda()
    mask_id = V - 1
    ya = torch.zeros(rows, dtype=torch.int32, device="cuda")
    ca = torch.zeros(rows, device="cuda")
    yb, cb = torch.full_like(ya, -5), torch.full_like(ca, -5.0)
    scratch = torch.empty(rows * 512, dtype=torch.uint8, device="cuda")
    Bd.polestar_k_confidence(logits, mask_id, ya, ca, scratch)
    Bd.polestar_k_confidence_noalloc(logits, mask_id, yb, cb)
    torch.cuda.synchronize()
    assert torch.equal(ya, yb)
    assert np.allclose(ca.cpu().numpy(), cb.cpu().numpy(), rtol=1e-4, atol=1e-7)
    assert (cb > 0).all() and (cb <= 1.0 + 1e-6).all()


def test_noalloc_matches_scratch_version_twice_in_a_row():
    # two calls back to back, the second with a different (smaller) shape: stale partials of the
    # first call stay in the built-in array and must not leak into the second result
    _run_pair(64, 126464, seed=1)
    _run_pair(5, 1000, seed=2)
    _run_pair(64, 126464, seed=3)


def test_noalloc_rejects_more_rows_than_its_scratch_holds():
    rows = Bd.NOALLOC_MAX_ROWS + 1
    logits = torch.zeros((rows, 8), device="cuda")
    y = torch.zeros(rows, dtype=torch.int32, device="cuda")
    c = torch.zeros(rows, device="cuda")
    with pytest.raises(Bd.PolestarError) as e:
        Bd.polestar_k_confidence_noalloc(logits, 7, y, c)
    assert e.value.code == Bd.E_NOSPACE
