"""Forward of the vector-quantized record (4-D centroids with 8-bit indices, 2-D centroids with 6-bit indices) against the
fp64 oracle of Eq. 8; records are produced by the oracle's quantizer from seeded weights, or drawn at random at the larger
sizes."""
import numpy as np
import pytest
import torch

from oracle import lopro_oracle as o
from paper_2601_19675_b200 import lopro, synth
from tests._layers import bf16_bits_to_device, device_bf16_to_f64

pytestmark = pytest.mark.gpu


def _dev16(a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()


def _random_record(n, m, cb_rows, cb_cols, r, seed, dim=4):
    rng = np.random.Generator(np.random.Philox(key=[seed, 99]))
    k = 256 if dim == 4 else 64
    idx = rng.integers(0, k, size=(m, n // dim), dtype=np.uint8)
    n_rg, n_cg = -(-m // cb_rows), n // cb_cols
    books_bits = synth.f32_to_bf16_bits((rng.standard_normal((n_rg, n_cg, k, dim)) * 0.02).astype(np.float32))
    a_bits, b_bits = synth.factors(m, n, max(r, 1), seed=seed)
    return idx, books_bits, synth.permutation(n, seed=seed), a_bits[:, :r], b_bits[:r]


def _check(d, idx, books_bits, perm, a_bits, b_bits, T, seed, rows=None):
    blob = lopro.vq_pack(d, torch.from_numpy(idx).cuda(), _dev16(books_bits), torch.from_numpy(perm).cuda(),
                         _dev16(np.ascontiguousarray(a_bits)) if d.rank else None, _dev16(np.ascontiguousarray(b_bits)) if d.rank else None)
    x_bits = synth.activations(T, d.d_in, seed=seed, outlier_frac=0.01)
    x = bf16_bits_to_device(x_bits)
    ws = torch.zeros(lopro.vq_workspace_bytes(d, T), dtype=torch.uint8, device="cuda")
    y_bf = lopro.vq_linear_fwd(d, blob, x, lopro.OUT_BF16, workspace=ws).clone()
    y_f32 = lopro.vq_linear_fwd(d, blob, x, lopro.OUT_F32, workspace=ws)
    torch.cuda.synchronize()
    assert lopro.workspace_status(ws) == lopro.OK
    sel = slice(None) if rows is None else rows
    dim = d.dim if d.dim else 4
    x64 = o.bf16_bits_to_f64(x_bits)
    books = o.bf16_bits_to_f64(books_bits)
    a = o.f16_bits_to_f64(a_bits)[sel] if d.rank else np.zeros((len(idx[sel]), 0))
    b = o.f16_bits_to_f64(b_bits) if d.rank else np.zeros((0, d.d_in))
    # the oracle on the selected rows: their indices, and the codebooks of the groups they fall in
    if rows is None:
        exact = o.forward_exact_vq(x64, idx, books, perm, a, b, dim, d.cb_rows, d.cb_cols, d.identity_cols, d.block_size)
        w_hat = o.vq_dequant(idx, books, dim, d.cb_rows, d.cb_cols)
    else:
        w_hat = np.stack([o.vq_dequant(idx[r:r + 1], books[r // d.cb_rows:r // d.cb_rows + 1], dim, d.cb_rows, d.cb_cols)[0] for r in rows])
        exact = o.rotate(x64, perm, d.identity_cols, d.block_size) @ w_hat.T + (x64 @ b.T) @ a.T
    # declared roundings of the kernel: x~ to bf16, t to fp16 (centroids are bf16 already); fp32 accumulation
    xt = o.round_bf16(o.rotate(x64, perm, d.identity_cols, d.block_size))
    mirrored = xt @ w_hat.T + (o.round_f16(x64 @ b.T) @ a.T if d.rank else 0.0)
    got_bf = device_bf16_to_f64(y_bf)[:, sel]
    got_f32 = y_f32.cpu().numpy().astype(np.float64)[:, sel]
    assert o.max_rel_err(got_bf, exact) <= 2e-2
    assert o.max_rel_err(got_f32, mirrored) <= 1e-3
    assert np.array_equal(got_bf, o.round_bf16(got_f32))


@pytest.mark.parametrize("T", [1, 5, 8, 16, 31, 32, 40, 100])
@pytest.mark.parametrize("n,m,cr,cc,b,r", [(512, 128, 64, 256, 64, 16), (1024, 192, 128, 256, 128, 5), (768, 64, 64, 128, 256, 0)])
def test_vq_forward_random_records(T, n, m, cr, cc, b, r):
    d = lopro.make_vq_desc(n, m, cr, cc, b, rank=r)
    _check(d, *_random_record(n, m, cr, cc, r, seed=T + n), T=T, seed=T)


@pytest.mark.parametrize("T", [1, 5, 8, 16, 31, 32, 40, 100])
@pytest.mark.parametrize("n,m,cr,cc,b,r", [(512, 128, 64, 256, 64, 16), (1024, 192, 128, 256, 128, 5), (768, 64, 64, 128, 256, 0),
                                           (4096, 64, 64, 64, 128, 0)])
def test_vq_forward_random_records_with_two_dimensional_centroids(T, n, m, cr, cc, b, r):
    # the 3-bit form: 64 centroids of two entries per group, 6-bit indices packed by lopro_vq_pack (the last shape has 64
    # codebooks per row group: two sections of 32 pass through shared memory)
    d = lopro.make_vq_desc(n, m, cr, cc, b, rank=r, dim=2)
    assert lopro.vq_packed_bytes(d) < lopro.vq_packed_bytes(lopro.make_vq_desc(n, m, cr, cc, b, rank=r)) * 1.6
    _check(d, *_random_record(n, m, cr, cc, r, seed=T + n, dim=2), T=T, seed=T)


def test_vq_forward_of_a_3_bit_record_quantized_by_the_oracle():
    n, m, cr, cc, b, r, T = 512, 256, 128, 256, 64, 16, 8
    w = synth.weights(m, n, seed=3, spikes=20).astype(np.float64)
    perm = synth.permutation(n, seed=4)
    u, sig, v = o.svd_lowrank(w, r)
    a, bb = o.round_f16(u * sig[None, :]), o.round_f16(v)
    rp = o.partial_block_rotate(o.permute_columns(w - a @ bb, perm), b, b)
    rng = np.random.Generator(np.random.Philox(key=[7, 8]))
    picks = [[rng.integers(0, cr * cc // 2, size=64) for _ in range(n // cc)] for _ in range(m // cr)]
    idx, books = o.vq_quantize(rp, 2, 6, cr, cc, picks)
    d = lopro.make_vq_desc(n, m, cr, cc, b, rank=r, dim=2)
    _check(d, idx.astype(np.uint8), o.f64_to_bf16_bits(books), perm, o.f64_to_f16_bits(a), o.f64_to_f16_bits(bb), T=T, seed=5)
    # an index beyond the 64 centroids is rejected
    bad = idx.astype(np.uint8).copy()
    bad[5, 7] = 64
    with pytest.raises(lopro.LoproError) as e:
        lopro.vq_pack(d, torch.from_numpy(bad).cuda(), _dev16(o.f64_to_bf16_bits(books)), torch.from_numpy(perm).cuda(),
                      _dev16(o.f64_to_f16_bits(a)), _dev16(o.f64_to_f16_bits(bb)))
    assert e.value.status == lopro.ERR_INVALID_DATA


def test_vq_forward_of_a_record_quantized_by_the_oracle():
    # weights -> rank-16 part by SVD, residual rotated, vector-quantized with a randomly initialised codebook (oracle);
    # the record is packed and run: the output approximates W x as the oracle's own forward of the record does
    n, m, cr, cc, b, r, T = 512, 256, 128, 256, 64, 16, 8
    w = synth.weights(m, n, seed=3, spikes=20).astype(np.float64)
    perm = synth.permutation(n, seed=4)
    u, sig, v = o.svd_lowrank(w, r)
    a, bb = o.round_f16(u * sig[None, :]), o.round_f16(v)
    rp = o.partial_block_rotate(o.permute_columns(w - a @ bb, perm), b, b)
    rng = np.random.Generator(np.random.Philox(key=[7, 7]))
    picks = [[rng.integers(0, cr * cc // 4, size=256) for _ in range(n // cc)] for _ in range(m // cr)]
    idx, books = o.vq_quantize(rp, 4, 8, cr, cc, picks)
    d = lopro.make_vq_desc(n, m, cr, cc, b, rank=r)
    _check(d, idx.astype(np.uint8), o.f64_to_bf16_bits(books), perm, o.f64_to_f16_bits(a), o.f64_to_f16_bits(bb), T=T, seed=5)


@pytest.mark.parametrize("T", [1, 16])
def test_vq_forward_at_the_size_of_a_decoder_projection(T):
    # 4096 -> 11008, codebooks of 512 x 256 (0.125 bit per weight), block 256, rank 16: sampled rows
    n, m, cr, cc, b, r = 4096, 11008, 512, 256, 256, 16
    d = lopro.make_vq_desc(n, m, cr, cc, b, rank=r)
    rows = np.unique(np.concatenate([[0, 15, 16, 63, 64, 511, 512, m - 1], np.random.default_rng(T).integers(0, m, size=24)]))
    _check(d, *_random_record(n, m, cr, cc, r, seed=T), T=T, seed=T + 1, rows=rows)


def test_vq_pack_rejects_a_bad_permutation_and_the_record_stays_harmless():
    n, m = 512, 64
    d = lopro.make_vq_desc(n, m, 64, 256, 64, rank=0)
    idx, books_bits, perm, _, _ = _random_record(n, m, 64, 256, 0, seed=1)
    bad = perm.copy()
    bad[3] = bad[4]
    with pytest.raises(lopro.LoproError) as e:
        lopro.vq_pack(d, torch.from_numpy(idx).cuda(), _dev16(books_bits), torch.from_numpy(bad).cuda())
    assert e.value.status == lopro.ERR_INVALID_DATA
    bad[3] = n + 100
    with pytest.raises(lopro.LoproError) as e:
        lopro.vq_pack(d, torch.from_numpy(idx).cuda(), _dev16(books_bits), torch.from_numpy(bad).cuda())
    assert e.value.status == lopro.ERR_INVALID_DATA
    assert lopro.vq_packed_bytes(lopro.make_vq_desc(500, 64, 64, 256, 64)) == 0          # d_in not a multiple of 64
