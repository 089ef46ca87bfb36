"""The paper-format low-rank record (U, V in fp8 e4m3, Sigma and s in fp16; Sec. 3.3, Algorithm 1's saved record,
Appendix A.2): pack / unpack bit-exact, forward against the fp64 oracle y = U (Sigma (V (x / s))) + W^ Q^T P^T x."""
import numpy as np
import pytest
import torch

from oracle import lopro_oracle as o
from paper_2601_19675_b200 import lopro, synth
from tests._layers import bf16_bits_to_device, device_bf16_to_f64, random_layer_np
from tests.test_gpu_forward import _gate_b_with_ties

pytestmark = pytest.mark.gpu


def _dev(a):
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(a).cuda()


def _pack(d, layer, rec):
    return lopro.pack_lr8(d, _dev(layer["codes"]), _dev(layer["scales"]), _dev(layer["zeros"]), _dev(layer["perm"]),
                          _dev(rec["U"]), _dev(rec["V"]), _dev(rec["sigma"]), _dev(rec["s"]))


def _oracle_args(layer, rec, d, rows=None):
    sel = slice(None) if rows is None else np.asarray(rows)
    return dict(codes=layer["codes"][sel], scales=o.f16_bits_to_f64(layer["scales"])[sel], zeros=o.f16_bits_to_f64(layer["zeros"])[sel],
                perm=layer["perm"], u=o.e4m3_bits_to_f64(rec["U"])[sel], sigma=o.f16_bits_to_f64(rec["sigma"]),
                v=o.e4m3_bits_to_f64(rec["V"]), s=o.f16_bits_to_f64(rec["s"]), g=d.group_size, b_i=d.identity_cols, b_h=d.block_size)


def _gate_b_with_t_ties(x64, folded, mirrored, got_f32):
    """Gate B when an entry of t = B x sits on an fp16 rounding boundary.  The kernel adds the products of a row of B
    in fp32 (tile by tile), the oracle in fp64; an entry of the exact t within the fp32 summation error of the midpoint
    of two fp16 values (here: 64 * 2^-24 * sum_k |B[j,k] x[k]|) may round to either side, which moves the token's
    outputs by (other - chosen) * A[:, j] -- visible where the rank-r term dominates y.  Everything here comes from the
    oracle; a flip is kept only if it lowers the token's error (greedy witness search, as for the bf16 ties of the
    rotated activations)."""
    a, b = folded["a"], folded["b"]
    t_exact = x64 @ b.T
    slack = 64.0 * 2.0 ** -24 * (np.abs(x64) @ np.abs(b).T)
    chosen = o.round_f16(t_exact)
    step = np.maximum(np.abs(chosen), 2.0 ** -14) * 2.0 ** -10
    other = np.where(t_exact > chosen, o.round_f16(chosen + step), np.where(t_exact < chosen, o.round_f16(chosen - step), chosen))
    near = (other != chosen) & (np.abs(t_exact - 0.5 * (chosen + other)) <= slack)
    worst = 0.0
    for tok in range(x64.shape[0]):
        y = mirrored[tok].copy()
        best = o.max_rel_err(got_f32[tok:tok + 1], y[None, :])
        for j in np.flatnonzero(near[tok]):
            y_alt = y + (other[tok, j] - chosen[tok, j]) * a[:, j]
            e = o.max_rel_err(got_f32[tok:tok + 1], y_alt[None, :])
            if e < best:
                y, best = y_alt, e
        worst = max(worst, best)
    return worst


def _check(d, layer, rec, x_bits, rows=None):
    blob = _pack(d, layer, rec)
    x = bf16_bits_to_device(x_bits)
    T = x.shape[0]
    ws = torch.zeros(lopro.workspace_bytes(d, T), dtype=torch.uint8, device="cuda")
    y_bf = lopro.linear_fwd(d, blob, x, lopro.OUT_BF16, workspace=ws)
    y_f32 = lopro.linear_fwd(d, blob, x, lopro.OUT_F32, workspace=ws)
    torch.cuda.synchronize()
    assert lopro.workspace_status(ws) == lopro.OK
    args = _oracle_args(layer, rec, d, rows)
    x64 = o.bf16_bits_to_f64(x_bits)
    exact = o.forward_exact_unfolded(x64, **args)
    if lopro.linear_fwd_path(d, T)[0] == lopro.PATH_PREFILL:
        # tensor-core path: the record is folded into fp16 factors first, A = U Sigma and B = V / s (one rounding each),
        # and the dequantized weights are rounded to bf16
        folded = {k: args[k] for k in ("codes", "scales", "zeros", "perm", "g", "b_i", "b_h")}
        folded.update(a=o.round_f16(args["u"] * args["sigma"][None, :]), b=o.round_f16(args["v"] / args["s"][None, :]))
        mirrored = o.forward_mirrored(x64, **folded, round_w=True, round_t="f16", out="f32")
    else:
        folded = None
        mirrored = o.forward_mirrored_unfolded(x64, **args, round_t="f16", out="f32")
    got_bf, got_f32 = device_bf16_to_f64(y_bf), y_f32.cpu().numpy().astype(np.float64)
    if rows is not None:
        got_bf, got_f32 = got_bf[:, rows], got_f32[:, rows]
    assert o.max_rel_err(got_bf, exact) <= 2e-2
    err_b = o.max_rel_err(got_f32, mirrored)
    if err_b > 1e-3 and folded is not None:
        # a rotated entry within rounding distance of a bf16 tie may go to either side (see test_gpu_forward)
        err_b = _gate_b_with_ties(x64, folded, True, mirrored, got_f32)
    if err_b > 1e-3 and folded is not None:
        err_b = _gate_b_with_t_ties(x64, folded, mirrored, got_f32)
    assert err_b <= 1e-3
    # the low-rank branch is not negligible in these layers: dropping it would fail the gate
    no_lr = dict(args, sigma=np.zeros_like(args["sigma"]))
    assert o.max_rel_err(o.forward_exact_unfolded(x64, **no_lr), exact) > 5e-2


@pytest.mark.parametrize("n,m,bits,g,r", [(512, 272, 4, 128, 16), (1024, 48, 2, 64, 33)])
def test_pack_unpack_of_the_fp8_record_is_bit_exact(n, m, bits, g, r):
    layer = random_layer_np(n, m, bits, g, 0, seed=2)
    rec = synth.lowrank_record(m, n, r, seed=2)
    d = lopro.make_desc(n, m, bits, g, 64, rank=r, lowrank_format=lopro.LOWRANK_FP8)
    blob = _pack(d, layer, rec)
    back = lopro.unpack_lr8(d, blob)
    for k in ("U", "V", "sigma", "s"):
        assert np.array_equal(back[k].cpu().numpy().view(np.uint8).reshape(-1), np.ascontiguousarray(rec[k]).view(np.uint8).reshape(-1)), k
    out = lopro.unpack(d, blob)
    assert np.array_equal(out["codes"].cpu().numpy(), layer["codes"]) and "A" not in out
    assert np.array_equal(out["words"].cpu().numpy().view(np.uint32), o.pack_canonical(layer["codes"], bits))
    # storage accounting (Appendix A.2 with d_r = 8): one byte per factor entry
    assert lopro.packed_section(d, lopro.SEC_A)[1] == m * ((r + 15) // 16 * 16)
    assert lopro.packed_section(d, lopro.SEC_B)[1] == ((r + 15) // 16 * 16) * n
    # rejected: NaN pattern in U, zero in s; the folded entry point refuses an FP8 descriptor
    bad = dict(rec, U=rec["U"].copy()); bad["U"][3, 1] = 0x7F
    with pytest.raises(lopro.LoproError) as e:
        _pack(d, layer, bad)
    assert e.value.status == lopro.ERR_INVALID_DATA
    bad = dict(rec, s=rec["s"].copy()); bad["s"][7] = 0
    with pytest.raises(lopro.LoproError) as e:
        _pack(d, layer, bad)
    assert e.value.status == lopro.ERR_INVALID_DATA
    with pytest.raises(lopro.LoproError) as e:
        lopro.pack(d, _dev(layer["codes"]), _dev(layer["scales"]), _dev(layer["zeros"]), _dev(layer["perm"]))
    assert e.value.status == lopro.ERR_INVALID_ARG


def test_cfg1_layer_quantized_by_the_oracle_with_fp8_factors():
    # configuration 1 (512 x 512, 16 tokens, 4-bit g128, b_I = b_H = 64, rank 16) quantized as Algorithm 1 does: R1SVD
    # with the e4m3 casts inside the loop, activation scale s kept apart, RTN on the permuted-and-rotated residual
    c = synth.CONFIGS["cfg1"]
    n, m, r = c["d_in"], c["d_out"], c["rank"]
    w = synth.weights(m, n, seed=0)
    perm = synth.permutation(n, seed=0)
    s = o.f16_bits_to_f64(synth.lowrank_record(m, n, r, seed=0)["s"])
    q = o.lopro_quantize_unfolded(w, perm, c["identity_cols"], c["block_size"], r, c["bits"], c["group_size"], s, it=8,
                                  sketches=synth.sketches(r, n, seed=0))
    layer = dict(codes=q["codes"], scales=o.f64_to_f16_bits(q["scales"]), zeros=o.f64_to_f16_bits(q["zeros"]), perm=perm)
    rec = dict(U=o.f64_to_e4m3_bits(q["U"]), V=o.f64_to_e4m3_bits(q["V"]), sigma=o.f64_to_f16_bits(q["sigma"]),
               s=o.f64_to_f16_bits(q["s"]))
    d = lopro.make_desc(n, m, c["bits"], c["group_size"], c["block_size"], c["identity_cols"], r, lowrank_format=lopro.LOWRANK_FP8)
    x_bits = synth.activations(16, n, seed=0)
    blob = _pack(d, layer, rec)
    x = bf16_bits_to_device(x_bits)
    y_f32 = lopro.linear_fwd(d, blob, x, lopro.OUT_F32).cpu().numpy().astype(np.float64)
    y_bf = device_bf16_to_f64(lopro.linear_fwd(d, blob, x, lopro.OUT_BF16))
    args = _oracle_args(layer, rec, d)
    x64 = o.bf16_bits_to_f64(x_bits)
    assert o.max_rel_err(y_bf, o.forward_exact_unfolded(x64, **args)) <= 2e-2
    assert o.max_rel_err(y_f32, o.forward_mirrored_unfolded(x64, **args)) <= 1e-3
    # and the quantized layer approximates the dense one
    dense = x64 @ w.astype(np.float64).T
    assert np.linalg.norm(y_bf - dense) / np.linalg.norm(dense) < 0.12


def _tall_rows(tiles_per_sm, extra):
    return 16 * (torch.cuda.get_device_properties(0).multi_processor_count * tiles_per_sm + extra)


@pytest.mark.parametrize("T", [1, 3, 8, 16, 32, 40, 100])
@pytest.mark.parametrize("bits,g,r,m", [(4, 128, 32, 272), (2, 64, 128, 144), (3, 64, 17, None)])
def test_forward_with_the_fp8_record(T, bits, g, r, m):
    # the 32-warp, the 16-warp and the persistent small-batch kernel, and more than 32 tokens as chunks of 32
    n = 2048
    m = _tall_rows(3, 5) if m is None else m
    layer = random_layer_np(n, m, bits, g, 0, seed=T + bits)
    rec = synth.lowrank_record(m, n, r, seed=T + r)
    # Sigma large enough for the rank-r term to matter next to the synthetic quantized part
    rec["sigma"] = synth.f32_to_f16_bits(np.float32(40.0) * o.f16_bits_to_f64(rec["sigma"]).astype(np.float32))
    d = lopro.make_desc(n, m, bits, g, 128, rank=r, lowrank_format=lopro.LOWRANK_FP8)
    path, launches = lopro.linear_fwd_path(d, T)
    assert path in (lopro.PATH_WIDE, lopro.PATH_STREAM, lopro.PATH_TALL) or (T > 32 and path == lopro.PATH_PREFILL)
    if T > 32 and path != lopro.PATH_PREFILL:
        assert launches == 1 + (T + 31) // 32
    rows = None if m * n <= 1 << 21 else np.arange(0, m, 5)
    _check(d, layer, rec, synth.activations(T, n, seed=T + 1, outlier_frac=0.01), rows=rows)


@pytest.mark.parametrize("n,m,bits,g,r,T", [(1024, 256, 4, 128, 16, 300), (2048, 400, 3, 64, 33, 130), (1024, 384, 2, 64, 128, 700)])
def test_many_tokens_with_the_fp8_record_run_on_the_tensor_core_kernels(n, m, bits, g, r, T):
    # the record is folded into fp16 factors in the workspace (one more launch), then the same kernels as for a folded layer
    layer = random_layer_np(n, m, bits, g, 0, seed=T + bits)
    rec = synth.lowrank_record(m, n, r, seed=T + r)
    rec["sigma"] = synth.f32_to_f16_bits(np.float32(40.0) * o.f16_bits_to_f64(rec["sigma"]).astype(np.float32))
    d = lopro.make_desc(n, m, bits, g, 128, rank=r, lowrank_format=lopro.LOWRANK_FP8)
    x_bits = synth.activations(T, n, seed=T + 1, outlier_frac=0.01)
    with lopro.configured(lopro.OPT_NO_CHUNKS, 1):
        assert lopro.linear_fwd_path(d, T)[0] == lopro.PATH_PREFILL
        _check(d, layer, rec, x_bits)
        with lopro.configured(lopro.OPT_NO_CTA_PAIRS, 1):
            _check(d, layer, rec, x_bits)
    # the library's own choice (chunks of 32 tokens or the tensor-core kernels) agrees with the oracle as well
    _check(d, layer, rec, x_bits)


def test_large_layer_with_the_fp8_record_and_its_byte_saving():
    # configuration 4 (8192 -> 28672, 2-bit g64, block 256, rank 128) at 16 tokens: fp8 factors take half the bytes of
    # the folded fp16 ones -- 4.7 MB of 84 MB per forward
    c = synth.CONFIGS["cfg4"]
    n, m, r = c["d_in"], c["d_out"], c["rank"]
    layer = random_layer_np(n, m, c["bits"], c["group_size"], 0, seed=4)
    rec = synth.lowrank_record(m, n, r, seed=4)
    rec["sigma"] = synth.f32_to_f16_bits(np.float32(40.0) * o.f16_bits_to_f64(rec["sigma"]).astype(np.float32))
    d8 = lopro.make_desc(n, m, c["bits"], c["group_size"], c["block_size"], c["identity_cols"], r, lowrank_format=lopro.LOWRANK_FP8)
    d16 = lopro.make_desc(n, m, c["bits"], c["group_size"], c["block_size"], c["identity_cols"], r)
    saved = lopro.packed_bytes(d16) - lopro.packed_bytes(d8)
    assert abs(saved - (r * (m + n) - 2 * r - 2 * n)) <= 4 * 256      # one byte per factor entry less, Sigma and s added
    rows = np.unique(np.concatenate([[0, 15, 16, m - 1], np.random.default_rng(4).integers(0, m, size=24)]))
    _check(d8, layer, rec, synth.activations(16, n, seed=5), rows=rows)
