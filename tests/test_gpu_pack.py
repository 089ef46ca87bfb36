"""GPU parity of lopro_pack / lopro_unpack with the oracle's canonical bit stream: bit-exact."""
import numpy as np
import pytest
import torch

from oracle import lopro_oracle as o
from paper_2601_19675_b200 import lopro, synth
from tests._layers import random_layer_np, to_device

pytestmark = pytest.mark.gpu

CASES = [
    # d_in, d_out, bits, g, rank
    (512, 512, 4, 128, 16),
    (256, 48, 3, 64, 5),
    (1024, 272, 2, 64, 0),
    (11008 // 43 * 3, 144, 3, 128, 33),   # n = 768
    (4096, 4096, 4, 128, 32),
]


def _same_bits(t, ref_np):
    got = t.cpu().numpy()
    ref = np.ascontiguousarray(ref_np)
    return np.array_equal(got.view(np.uint8).reshape(-1), ref.view(np.uint8).reshape(-1))


@pytest.mark.parametrize("n,m,bits,g,r", CASES)
@pytest.mark.parametrize("layout", [lopro.LAYOUT_CANONICAL, lopro.LAYOUT_FRAGMENT, lopro.LAYOUT_ROWBLOCK])
def test_pack_unpack_bit_exact(n, m, bits, g, r, layout):
    layer = random_layer_np(n, m, bits, g, r, seed=3)
    dev = to_device(layer)
    d = lopro.make_desc(n, m, bits, g, 64, rank=r, layout=layout)
    blob = lopro.pack(d, dev["codes"], dev["scales"], dev["zeros"], dev["perm"], dev["A"], dev["B"])
    words_ref = o.pack_canonical(layer["codes"], bits)
    if layout == lopro.LAYOUT_CANONICAL:
        off, nbytes = lopro.packed_section(d, lopro.SEC_CODES)
        assert _same_bits(blob[off:off + nbytes], words_ref)       # the stored bytes ARE the canonical stream
    out = lopro.unpack(d, blob)
    assert _same_bits(out["words"], words_ref)
    assert _same_bits(out["codes"], layer["codes"])
    assert np.array_equal(out["codes"].cpu().numpy(), o.unpack_canonical(out["words"].cpu().numpy().view(np.uint32), bits, n))
    assert _same_bits(out["scales"], layer["scales"])
    assert _same_bits(out["zeros"], layer["zeros"])
    assert _same_bits(out["perm"], layer["perm"])
    if r:
        assert _same_bits(out["A"], layer["A"])
        assert _same_bits(out["B"], layer["B"])
    # equal layers give equal blobs (padding is zeroed)
    blob2 = lopro.pack(d, dev["codes"], dev["scales"], dev["zeros"], dev["perm"], dev["A"], dev["B"])
    assert torch.equal(blob, blob2)


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("layout", [lopro.LAYOUT_FRAGMENT, lopro.LAYOUT_ROWBLOCK])
def test_walking_patterns_roundtrip(bits, layout):
    # every code value at every position of a 16 x 64 tile, one at a time in a field of the complement
    n, m, g = 64, 16, 64
    qmax = 2 ** bits - 1
    d = lopro.make_desc(n, m, bits, g, 64, rank=0, layout=layout)
    ones = np.full((m, n // g), 0x3C00, dtype=np.uint16)
    perm = torch.arange(n, dtype=torch.int32, device="cuda")
    sc = torch.from_numpy(ones.view(np.int16)).cuda()
    for pos in range(0, m * n, 37):
        codes = np.zeros((m, n), dtype=np.uint8)
        codes.reshape(-1)[pos] = qmax
        codes.reshape(-1)[(pos * 7 + 11) % (m * n)] = 1
        blob = lopro.pack(d, torch.from_numpy(codes).cuda(), sc, sc, perm)
        out = lopro.unpack(d, blob, want=("codes", "words"))
        assert np.array_equal(out["codes"].cpu().numpy(), codes)
        assert np.array_equal(out["words"].cpu().numpy().view(np.uint32), o.pack_canonical(codes, bits))


def test_pack_rejects_invalid_layer_data():
    n, m, bits, g, r = 256, 32, 3, 64, 4
    layer = random_layer_np(n, m, bits, g, r, seed=5)
    d = lopro.make_desc(n, m, bits, g, 64, rank=r)

    def try_pack(**override):
        L = dict(layer)
        L.update(override)
        dev = to_device(L)
        return lopro.pack(d, dev["codes"], dev["scales"], dev["zeros"], dev["perm"], dev["A"], dev["B"])

    try_pack()
    bad = layer["codes"].copy(); bad[7, 100] = 8
    with pytest.raises(lopro.LoproError) as e:
        try_pack(codes=bad)
    assert e.value.status == lopro.ERR_INVALID_DATA
    bad = layer["perm"].copy(); bad[3] = bad[4]
    with pytest.raises(lopro.LoproError):
        try_pack(perm=bad)
    bad = layer["perm"].copy(); bad[0] = n
    with pytest.raises(lopro.LoproError):
        try_pack(perm=bad)
    bad = layer["scales"].copy(); bad[1, 1] = 0x7C00           # +inf
    with pytest.raises(lopro.LoproError):
        try_pack(scales=bad)
    bad = layer["scales"].copy(); bad[0, 0] = 0                # zero scale
    with pytest.raises(lopro.LoproError):
        try_pack(scales=bad)
    bad = layer["zeros"].copy(); bad[2, 3] = 0x7E00            # NaN
    with pytest.raises(lopro.LoproError):
        try_pack(zeros=bad)
    # the context is still usable and a clean pack still succeeds
    try_pack()
    # undersized blob
    dev = to_device(layer)
    small = torch.empty(lopro.packed_bytes(d) - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(lopro.LoproError) as e:
        lopro.pack(d, dev["codes"], dev["scales"], dev["zeros"], dev["perm"], dev["A"], dev["B"], out=small)
    assert e.value.status == lopro.ERR_BUFFER_TOO_SMALL


def test_unpack_rejects_mismatched_descriptor():
    n, m, bits, g, r = 256, 32, 4, 64, 0
    layer = random_layer_np(n, m, bits, g, r, seed=6)
    dev = to_device(layer)
    d = lopro.make_desc(n, m, bits, g, 64, rank=r)
    blob = lopro.pack(d, dev["codes"], dev["scales"], dev["zeros"], dev["perm"])
    d2 = lopro.make_desc(n, m, bits, g, 32, rank=r)
    with pytest.raises(lopro.LoproError) as e:
        lopro.unpack(d2, blob)
    assert e.value.status == lopro.ERR_INVALID_DATA


def test_a_rejected_blob_holds_no_out_of_range_index():
    # a permutation with entries outside [0, n) is rejected, and what is left in the blob cannot send a forward
    # out of bounds: the permutation section reads back all zeros (checked on the host; no forward is run on it)
    n, m, bits, g, r = 512, 64, 4, 128, 0
    layer = random_layer_np(n, m, bits, g, r, seed=8)
    d = lopro.make_desc(n, m, bits, g, 64, rank=r)
    bad = layer["perm"].copy()
    bad[5], bad[77] = n + 1000, -3
    dev = to_device(dict(layer, perm=bad))
    blob = torch.full((lopro.packed_bytes(d),), 0xFF, dtype=torch.uint8, device="cuda")
    with pytest.raises(lopro.LoproError) as e:
        lopro.pack(d, dev["codes"], dev["scales"], dev["zeros"], dev["perm"], out=blob)
    assert e.value.status == lopro.ERR_INVALID_DATA
    perm_back = lopro.perm_of(d, blob).cpu().numpy()
    assert perm_back.min() >= 0 and perm_back.max() < n
