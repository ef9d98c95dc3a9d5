"""bwla_w1ax_linear_static: the layer for callers that cannot allocate scratch memory.

A plug-in slot, a stage behind a frozen memory pool or a serving loop that may not call cudaMalloc has only its
input and output buffers; the entry point under test keeps its intermediates in an array built into the library.
Here it is called through the C ABI twice in a row, with different inputs, and each result must equal what the
ordinary entry point (caller-supplied workspace) gives for the same inputs, within the tolerance the parity
tests use for two runs of the same arithmetic: the outputs must be bit-identical, since both routes run the same
kernels.  The file sorts last so that every other test has run before it.
"""
import numpy as np
import pytest
import torch

from paper_2605_00422_b200 import inputs as gen
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_matches_workspace_entry_twice_in_a_row():
    from paper_2605_00422_b200 import bwla
    bwla.bwla_force_path(bwla.BWLA_PATH_AUTO)
    shape = gen.CONFIG_SHAPES[2][0]                       # 5120 -> 8192, Kronecker 64 x 80, rank 64
    lay = gen.make_layer(2, shape, 6, direct_words=True)
    dl = H.DeviceLayer(lay, bwla)
    out_static = torch.empty(16, shape.N, dtype=torch.bfloat16, device="cuda")   # the caller owns input and output
    for call, M in enumerate((16, 5)):                    # the second call finds the first one's leftovers
        x = H.bf16_to_dev(gen.make_activations(2, shape, M, layer=call))
        ws = bwla.new_workspace(M, shape.K, shape.N, shape.r, 6)
        want = bwla.bwla_w1ax_linear(x, dl.P1, dl.P2, 6, dl.packed, dl.alpha, dl.U, dl.V, workspace=ws)
        assert bwla.bwla_check_status(ws) == 0
        got = bwla.bwla_w1ax_linear_static(x, dl.P1, dl.P2, 6, dl.packed, dl.alpha, dl.U, dl.V, out=out_static[:M])
        torch.cuda.synchronize()
        assert np.array_equal(H.bf16_to_host(got), H.bf16_to_host(want)), f"call {call}: outputs differ"


def test_static_scratch_entry_refuses_what_does_not_fit():
    from paper_2605_00422_b200 import bwla
    shape = gen.small_shape(1024, 64, 32, 32, 0, shape_id=77)
    lay = gen.make_layer(0, shape, 6)
    dl = H.DeviceLayer(lay, bwla)
    M = bwla.BWLA_STATIC_SCRATCH_BYTES // shape.K + 1     # the codes alone exceed the built-in array
    x = torch.zeros(M, shape.K, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bwla.BwlaError) as e:
        bwla.bwla_w1ax_linear_static(x, dl.P1, dl.P2, 6, dl.packed, dl.alpha)
    assert e.value.status == bwla.BWLA_ERR_STATIC_SCRATCH


def test_static_scratch_entry_refuses_bad_arguments_before_touching_the_stream():
    from paper_2605_00422_b200 import bwla
    shape = gen.small_shape(64, 16, 8, 8, 0)
    lay = gen.make_layer(0, shape, 6)
    dl = H.DeviceLayer(lay, bwla)
    x = H.bf16_to_dev(gen.make_activations(0, shape, 2))
    with pytest.raises(bwla.BwlaError) as e:
        bwla.bwla_w1ax_linear_static(x, dl.P1, dl.P2, 5, dl.packed, dl.alpha)                      # bits not in {4,6,8}
    assert e.value.status == bwla.BWLA_ERR_INVALID_ARG
    with pytest.raises(bwla.BwlaError) as e:
        bwla.bwla_w1ax_linear_static(x, dl.P1, dl.P2[:4, :4].contiguous(), 6, dl.packed, dl.alpha)  # K != n1*n2
    assert e.value.status == bwla.BWLA_ERR_INVALID_ARG
    out = bwla.bwla_w1ax_linear_static(x, dl.P1, dl.P2, 6, dl.packed, dl.alpha)                    # and a good call still works
    torch.cuda.synchronize()
    assert out.shape == (2, 16)
