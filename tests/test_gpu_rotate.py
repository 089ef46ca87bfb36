"""GPU parity of lopro_rotate with the oracle's x~ = Q^T P^T x (Eq. 5, Eq. 6, Eq. 8)."""
import numpy as np
import pytest
import torch

from oracle import lopro_oracle as o
from paper_2601_19675_b200 import lopro, synth
from tests._layers import bf16_bits_to_device, device_bf16_to_f64

pytestmark = pytest.mark.gpu


def _ulp_bf16(v):
    """Spacing of bf16 numbers at |v| (8-bit significand), floored at the smallest normal's spacing."""
    a = np.maximum(np.abs(v), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(a)) - 7)


def _run(n, b_i, b_h, T, seed=0, ldx=None, outlier_frac=0.0):
    x_bits = synth.activations(T, n, seed=seed, outlier_frac=outlier_frac)
    perm = synth.permutation(n, seed=seed)
    d = lopro.make_desc(n, 16, 4, 64, b_h, identity_cols=b_i)
    assert lopro.check_desc(d) == lopro.OK
    xd = bf16_bits_to_device(x_bits)
    if ldx is not None:
        buf = torch.zeros((T, ldx), dtype=torch.bfloat16, device="cuda")
        buf[:, :n] = xd
        xd = buf[:, :n]
    out = lopro.rotate(d, torch.from_numpy(perm).cuda(), xd)
    torch.cuda.synchronize()
    got = device_bf16_to_f64(out)
    exact = o.rotate(o.bf16_bits_to_f64(x_bits), perm, b_i, b_h)
    return got, exact, x_bits, perm


@pytest.mark.parametrize("n,b_i,b_h,T", [
    (512, 64, 64, 16), (4096, 128, 128, 8), (4096, 128, 128, 1), (8192, 256, 256, 3), (11008, 128, 128, 5),
    (11008, 0, 256, 2), (4096, 0, 4096 // 4, 2), (2048, 0, 512, 3), (1024, 512, 512, 2), (4096, 64, 64, 33),
    (704, 64, 128, 4), (128, 126, 2, 4), (192, 4, 4, 3), (256, 0, 8, 2), (320, 64, 16, 2), (384, 32, 32, 7),
])
def test_rotate_matches_oracle_within_one_bf16_ulp(n, b_i, b_h, T):
    got, exact, _, _ = _run(n, b_i, b_h, T, seed=n + b_h + T)
    ref = o.round_bf16(exact)
    # fp32 butterflies then one rounding: may differ from rounding the fp64 result by one bf16 ulp,
    # and only where the exact value sits next to a rounding boundary.
    assert np.all(np.abs(got - exact) <= 0.5001 * _ulp_bf16(exact) + 1e-6 * np.abs(exact).max())
    assert np.mean(got == ref) > 0.995
    # identity prefix is a pure gather: bit-exact
    assert np.array_equal(got[:, :b_i], ref[:, :b_i])


@pytest.mark.parametrize("n,b_i,b_h,T", [
    (4096, 128, 128, 16), (4096, 128, 128, 2048), (8192, 256, 256, 77), (11008, 128, 128, 21), (1024, 0, 16, 19),
    (2048, 32, 32, 40), (4096, 64, 64, 257), (512, 512, 64, 17), (1024, 16, 16, 30), (12288, 0, 256, 18), (14336, 256, 128, 16),
])
def test_rotate_many_rows_tensor_core_form(n, b_i, b_h, T):
    # 16 rows and more, b_H in 16..256, b_I a multiple of 16: the first four levels of the recursion as a product with
    # H_16 on the tensor cores (fp32 accumulation of sixteen +-x terms), the rest as fp32 add / subtract
    got, exact, _, _ = _run(n, b_i, b_h, T, seed=n + b_h + T, outlier_frac=0.01)
    ref = o.round_bf16(exact)
    assert np.all(np.abs(got - exact) <= 0.5001 * _ulp_bf16(exact) + 1e-6 * np.abs(exact).max())
    assert np.mean(got == ref) > 0.995
    assert np.array_equal(got[:, :b_i], ref[:, :b_i])


def test_pure_permutation_is_bit_exact_and_strided_rows_work():
    n, T = 4096, 9
    got, exact, x_bits, perm = _run(n, n, 128, T, seed=11, ldx=n + 64)
    assert np.array_equal(got, o.bf16_bits_to_f64(x_bits)[:, perm])
    got2, exact2, _, _ = _run(n, 128, 128, T, seed=11, ldx=n + 64)
    got3, _, _, _ = _run(n, 128, 128, T, seed=11)
    assert np.array_equal(got2, got3)
    got4, _, _, _ = _run(n, 128, 128, 37, seed=12, ldx=n + 64)          # many rows: the other kernel, strided as well
    got5, _, _, _ = _run(n, 128, 128, 37, seed=12)
    assert np.array_equal(got4, got5)


def test_rotation_preserves_norm_and_is_an_involution_on_the_device():
    # Q is symmetric and orthogonal (Eq. 6): applying the block rotation twice with the identity
    # permutation returns x up to two bf16 roundings; the norm is kept to bf16 accuracy.
    n, b, T = 4096, 128, 4
    x_bits = synth.activations(T, n, seed=21, outlier_frac=0.01)
    d = lopro.make_desc(n, 16, 4, 64, b, identity_cols=b)
    ident = torch.arange(n, dtype=torch.int32, device="cuda")
    x = bf16_bits_to_device(x_bits)
    once = lopro.rotate(d, ident, x)
    twice = lopro.rotate(d, ident, once)
    x64, t64, o64 = device_bf16_to_f64(x), device_bf16_to_f64(twice), device_bf16_to_f64(once)
    blocks = (x64.reshape(T, n // b, b), t64.reshape(T, n // b, b), o64.reshape(T, n // b, b))
    nx, no = np.linalg.norm(blocks[0], axis=2), np.linalg.norm(blocks[2], axis=2)
    assert np.allclose(nx, no, rtol=2e-3)
    assert np.all(np.linalg.norm(blocks[1] - blocks[0], axis=2) <= 1e-2 * nx + 1e-6)


def test_rotate_argument_errors():
    d = lopro.make_desc(512, 16, 4, 64, 64)
    perm = torch.arange(512, dtype=torch.int32, device="cuda")
    x = torch.zeros((4, 512), dtype=torch.bfloat16, device="cuda")
    out = torch.empty((0, 512), dtype=torch.bfloat16, device="cuda")
    lopro.rotate(d, perm, x[:0], out=out)                      # T = 0 is a no-op
    with pytest.raises(lopro.LoproError):
        lopro.rotate(d, perm, torch.zeros((4, 520), dtype=torch.bfloat16, device="cuda")[:, 4:516])  # misaligned rows
