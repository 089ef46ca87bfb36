"""lopro_linear_fwd_noalloc: the forward for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off the table -- inside a host application that
owns the device heap, or in a serving loop that cannot afford the device-wide synchronisation an
allocation may cause.  For them the library keeps its scratch in a fixed array of its own.  This test
calls that entry point through the C ABI twice in a row (the array is shared and keeps the previous
call's contents, so the second call proves nothing stale leaks into a result) and checks both
outputs against lopro_linear_fwd on the same inputs, with the tolerance of the forward tests; it
also checks that a request beyond the fixed array is refused cleanly.

Collected last on purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import lopro_oracle as o
from paper_2601_19675_b200 import lopro, synth
from tests._layers import bf16_bits_to_device, device_bf16_to_f64, random_layer_np, to_device

pytestmark = pytest.mark.gpu


def _layer(n, m, bits, g, b, r, seed, layout=lopro.LAYOUT_FRAGMENT):
    layer = random_layer_np(n, m, bits, g, r, seed=seed)
    d = lopro.make_desc(n, m, bits, g, b, rank=r, layout=layout)
    dev = to_device(layer)
    blob = lopro.pack(d, dev["codes"], dev["scales"], dev["zeros"], dev["perm"], dev["A"], dev["B"])
    return d, blob


def _two_calls(d, blob, n, m, token_counts):
    for call, T in enumerate(token_counts):     # second call: fewer tokens, other values, same shared scratch
        x = bf16_bits_to_device(synth.activations(T, n, seed=50 + call, outlier_frac=0.01))
        ref_bf = lopro.linear_fwd(d, blob, x, lopro.OUT_BF16)
        ref_f32 = lopro.linear_fwd(d, blob, x, lopro.OUT_F32)
        y_bf = torch.full((T, m), float("nan"), dtype=torch.bfloat16, device="cuda")
        y_f32 = torch.full((T, m), float("nan"), dtype=torch.float32, device="cuda")
        lopro.linear_fwd_noalloc(d, blob, x, y_bf, lopro.OUT_BF16)
        lopro.linear_fwd_noalloc(d, blob, x, y_f32, lopro.OUT_F32)
        torch.cuda.synchronize()
        # Both entry points launch the same kernels on the same inputs in the same fixed order, so the outputs
        # agree bit for bit -- a sharper check than the forward tests' tolerances (which it implies): anything
        # stale read from the shared scratch, or a misplaced offset inside it, would show.
        assert torch.isfinite(y_f32).all()
        assert torch.equal(y_bf, ref_bf)
        assert torch.equal(y_f32, ref_f32)
        assert o.max_rel_err(device_bf16_to_f64(y_bf), device_bf16_to_f64(ref_bf)) <= 2e-2
        assert o.max_rel_err(y_f32.cpu().numpy().astype(np.float64), ref_f32.cpu().numpy().astype(np.float64)) <= 1e-3


@pytest.mark.parametrize("layout", [lopro.LAYOUT_FRAGMENT, lopro.LAYOUT_ROWBLOCK])
@pytest.mark.parametrize("n,m,bits,g,b,r", [(1024, 272, 4, 128, 128, 16), (2048, 144, 2, 64, 256, 33)])
def test_two_calls_in_a_row_match_the_workspace_entry_point(n, m, bits, g, b, r, layout):
    # (row-block layout: blocks of rows shared between thread blocks leave arrival counters and partial sums in the
    # scratch; the counters must read zero again when the second call starts)
    d, blob = _layer(n, m, bits, g, b, r, seed=11, layout=layout)
    _two_calls(d, blob, n, m, (8, 3))


@pytest.mark.parametrize("no_chunks", [False, True])
def test_more_than_32_tokens_inside_the_fixed_scratch(no_chunks):
    # 40 and 33 tokens still fit the built-in array: as chunks of 32 through the small-batch kernels, and (with the
    # library's switch for it) through the tensor-core kernel
    n, m = 1024, 256
    d, blob = _layer(n, m, 4, 128, 128, 16, seed=13)
    with lopro.configured(lopro.OPT_NO_CHUNKS, 1 if no_chunks else 0):
        assert lopro.workspace_bytes(d, 40) <= lopro.NOALLOC_SCRATCH_BYTES
        assert (lopro.linear_fwd_path(d, 40)[0] == lopro.PATH_PREFILL) == no_chunks
        _two_calls(d, blob, n, m, (40, 33))


def test_requests_beyond_the_fixed_scratch_are_refused():
    n, m = 4096, 64
    d, blob = _layer(n, m, 4, 128, 128, 0, seed=12)
    T = 2048                                      # needs ~17 MB of scratch: more than the built-in array
    assert lopro.workspace_bytes(d, T) > lopro.NOALLOC_SCRATCH_BYTES
    x = torch.zeros((T, n), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((T, m), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lopro.LoproError) as e:
        lopro.linear_fwd_noalloc(d, blob, x, y)
    assert e.value.status == lopro.ERR_BUFFER_TOO_SMALL
    assert torch.count_nonzero(y) == 0            # nothing ran
    # T = 0 is a no-op, and a valid small request still works afterwards
    lopro.linear_fwd_noalloc(d, blob, x[:0], y[:0])
    lopro.linear_fwd_noalloc(d, blob, x[:4], y[:4])
    torch.cuda.synchronize()
