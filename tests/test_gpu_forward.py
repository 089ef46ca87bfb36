"""GPU parity of lopro_linear_fwd with the fp64 oracle of Eq. 8.

Gate A: bf16 output against the exact oracle, max relative error <= 2e-2.
Gate B: fp32 output (fp32 accumulation) against the mirrored oracle, which applies the roundings the
library declares (rotated activations to bf16, low-rank intermediate to fp16, and where the forward
runs the tensor-core prefill kernel the dequantized weights to bf16), <= 1e-3.
The error measure is oracle.max_rel_err (element-wise, relative to max(|y|, rms of the token's row))."""
import numpy as np
import pytest
import torch

from oracle import lopro_oracle as o
from paper_2601_19675_b200 import lopro, synth
from tests._layers import bf16_bits_to_device, device_bf16_to_f64, oracle_args, random_layer_np, to_device

pytestmark = pytest.mark.gpu

GATE_A = 2e-2
GATE_B = 1e-3


def _pack(layer, d):
    dev = to_device(layer)
    return lopro.pack(d, dev["codes"], dev["scales"], dev["zeros"], dev["perm"], dev["A"], dev["B"])


def _check_forward(layer, d, x_bits, rows=None, gate_a=GATE_A, gate_b=GATE_B):
    """Forward against the oracle on the path the library picks; where that is the chunked small-batch path
    (more than 32 tokens, few output rows) the tensor-core prefill path is checked as well."""
    T = x_bits.shape[0]
    res = _check_forward_once(layer, d, x_bits, rows, gate_a, gate_b)
    if d.layout == lopro.LAYOUT_FRAGMENT:
        # the same layer packed in the row-block layout: the tcgen05 small-batch kernel
        d2 = lopro.make_desc(d.d_in, d.d_out, d.bits, d.group_size, d.block_size, d.identity_cols, d.rank,
                             layout=lopro.LAYOUT_ROWBLOCK)
        assert lopro.linear_fwd_path(d2, T)[0] == lopro.PATH_ROWBLOCK
        _check_forward_once(layer, d2, x_bits, rows, gate_a, gate_b)
    if T > 32 and lopro.linear_fwd_path(d, T)[0] != lopro.PATH_PREFILL:
        with lopro.configured(lopro.OPT_NO_CHUNKS, 1):
            if lopro.linear_fwd_path(d, T)[0] == lopro.PATH_PREFILL:
                _check_forward_once(layer, d, x_bits, rows, gate_a, gate_b)
    return res


def _check_forward_once(layer, d, x_bits, rows, gate_a, gate_b):
    blob = _pack(layer, d)
    x = bf16_bits_to_device(x_bits)
    T = x.shape[0]
    # the tensor-core prefill kernel rounds the dequantized weights to bf16, the small-batch kernels do not
    round_w = lopro.linear_fwd_path(d, T)[0] == lopro.PATH_PREFILL
    ws = torch.zeros(lopro.workspace_bytes(d, T), dtype=torch.uint8, device="cuda")
    y_bf = lopro.linear_fwd(d, blob, x, lopro.OUT_BF16, workspace=ws)
    y_f32 = lopro.linear_fwd(d, blob, x, lopro.OUT_F32, workspace=ws)
    torch.cuda.synchronize()
    assert lopro.workspace_status(ws) == lopro.OK
    args = oracle_args(layer, d.group_size, d.identity_cols, d.block_size, rows=rows)
    x64 = o.bf16_bits_to_f64(x_bits)
    exact = o.forward_exact(x64, **args)
    mirrored = o.forward_mirrored(x64, **args, round_w=round_w, round_t="f16", out="f32")
    # declared roundings cannot hide an error: by themselves they stay inside gate A (rounding x~ to bf16 alone
    # reaches ~1 % on the max-over-entries measure once a layer has a few hundred thousand outputs)
    assert o.max_rel_err(mirrored, exact) <= GATE_A
    got_bf = device_bf16_to_f64(y_bf)
    got_f32 = y_f32.cpu().numpy().astype(np.float64)
    if rows is not None:
        got_bf, got_f32 = got_bf[:, rows], got_f32[:, rows]
    err_a = o.max_rel_err(got_bf, exact)
    err_b = o.max_rel_err(got_f32, mirrored)
    if err_b > gate_b:
        err_b = _gate_b_with_ties(x64, args, round_w, mirrored, got_f32)
    assert err_a <= gate_a, f"gate A: {err_a}"
    assert err_b <= gate_b, f"gate B: {err_b}"
    # bf16 output is the rounding of the fp32 output path (same accumulation order)
    assert np.array_equal(got_bf, o.round_bf16(got_f32))
    return err_a, err_b


def _gate_b_with_ties(x64, args, round_w, mirrored, got_f32):
    """Gate B when a rotated entry sits on a bf16 rounding boundary.  The kernels run the butterflies in fp32,
    the oracle in fp64; an entry of the exact x~ that lies within 1e-6 of its block's maximum of the midpoint
    between two bf16 values may legitimately round to either side (the rotation's own tolerance allows it).
    Everything here comes from the oracle: for each token with such entries the mirrored result is re-evaluated
    with such entries moved to the other side -- y is linear in x~, so flipping entry k of token t adds
    (other - chosen) * W^[:, k] -- and the token's outputs must meet the gate for one such choice."""
    b_i, b_h, g = args["b_i"], args["b_h"], args["g"]
    xt = o.rotate(x64, args["perm"], b_i, b_h)
    chosen = o.round_bf16(xt)
    # the neighbouring bf16 value on the other side of xt
    step = np.abs(chosen) * 2.0 ** -7
    other = np.where(xt > chosen, o.round_bf16(chosen + step), np.where(xt < chosen, o.round_bf16(chosen - step), chosen))
    mid = 0.5 * (chosen + other)
    n = xt.shape[1]
    blockmax = np.empty_like(xt)
    blockmax[:, :b_i] = np.abs(xt[:, :b_i])
    if n > b_i:
        bm = np.abs(xt[:, b_i:]).reshape(xt.shape[0], -1, b_h).max(axis=2, keepdims=True)
        blockmax[:, b_i:] = np.broadcast_to(bm, (xt.shape[0], (n - b_i) // b_h, b_h)).reshape(xt.shape[0], n - b_i)
    near = (other != chosen) & (np.abs(xt - mid) <= 1e-6 * blockmax)
    w_hat = o.dequant(args["codes"], args["scales"], args["zeros"], g)
    if round_w:
        w_hat = o.round_bf16(o.round_f32(w_hat))
    worst = 0.0
    for t in range(xt.shape[0]):
        # greedy search for a witness, largest rounding steps first: a flip is kept when it lowers the token's
        # error (a few entries per token qualify; only one with a large step can matter)
        ks = np.flatnonzero(near[t])
        ks = ks[np.argsort(-np.abs(other[t, ks] - chosen[t, ks]))]
        y = mirrored[t].copy()
        best = o.max_rel_err(got_f32[t:t + 1], y[None, :])
        for k in ks:
            y_alt = y + (other[t, k] - chosen[t, k]) * w_hat[:, k]
            e = o.max_rel_err(got_f32[t:t + 1], y_alt[None, :])
            if e < best:
                y, best = y_alt, e
        worst = max(worst, best)
    return worst


def test_cfg1_layer_quantized_by_the_oracle():
    # configuration 1: 512 x 512, 16 tokens, weights ~ N(0, 0.02) quantized by the oracle to 4-bit
    # asymmetric g = 128, random permutation, b_I = b_H = 64, rank 16.
    c = synth.CONFIGS["cfg1"]
    n, m, r = c["d_in"], c["d_out"], c["rank"]
    w = synth.weights(m, n, seed=0)
    perm = synth.permutation(n, seed=0)
    q = o.lopro_quantize(w, perm, c["identity_cols"], c["block_size"], r, c["bits"], c["group_size"], method="svd")
    layer = dict(codes=q["codes"], scales=o.f64_to_f16_bits(q["scales"]), zeros=o.f64_to_f16_bits(q["zeros"]),
                 perm=perm, A=o.f64_to_f16_bits(q["A"]), B=o.f64_to_f16_bits(q["B"]))
    d = lopro.make_desc(n, m, c["bits"], c["group_size"], c["block_size"], c["identity_cols"], r)
    x_bits = synth.activations(16, n, seed=0)
    _check_forward(layer, d, x_bits)
    # and the quantized layer approximates the dense one: y ~= W x (quantization error only)
    blob = _pack(layer, d)
    y = device_bf16_to_f64(lopro.linear_fwd(d, blob, bf16_bits_to_device(x_bits)))
    dense = o.bf16_bits_to_f64(x_bits) @ w.astype(np.float64).T
    assert np.linalg.norm(y - dense) / np.linalg.norm(dense) < 0.12


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("g", [64, 128])
@pytest.mark.parametrize("T", [1, 2, 3, 7, 8, 9, 15, 16, 17, 31, 32, 33, 65])
def test_token_count_edges(bits, g, T):
    n, m, r = 768, 144, 17                                    # ragged row tile (144 = 128 + 16), odd rank
    layer = random_layer_np(n, m, bits, g, r, seed=100 + bits + g)
    d = lopro.make_desc(n, m, bits, g, 128, identity_cols=128, rank=r)
    _check_forward(layer, d, synth.activations(T, n, seed=T))


@pytest.mark.parametrize("n,m,bits,g,b_i,b_h,r,T", [
    (64, 16, 4, 64, 0, 64, 0, 1),            # smallest layer, no low-rank branch
    (64, 16, 2, 64, 64, 2, 1, 5),            # rotation disabled (b_I = n)
    (1024, 256, 3, 256, 0, 1024, 64, 4),     # full-width Hadamard (the full-rotation ablation)
    (2048, 128, 4, 128, 0, 512, 8, 8),
    (4096, 512, 4, 128, 256, 256, 32, 8),    # several K slices and panels
    (8192, 256, 2, 64, 256, 256, 128, 16),
    (4096, 384, 3, 64, 128, 128, 64, 40),
    (11008, 128, 4, 128, 128, 128, 32, 2),   # the 7B 'down' projection width
])
def test_shapes_in_the_parameter_domain(n, m, bits, g, b_i, b_h, r, T):
    layer = random_layer_np(n, m, bits, g, r, seed=n + m + bits)
    d = lopro.make_desc(n, m, bits, g, b_h, identity_cols=b_i, rank=r)
    _check_forward(layer, d, synth.activations(T, n, seed=7, outlier_frac=0.01))


@pytest.mark.parametrize("n,m,bits,g,r,T", [
    (512, 320, 3, 64, 17, 512),      # one 512-token chunk; second row tile ragged (its second CTA has no rows at all)
    (1024, 256, 4, 128, 64, 600),    # 512 + 88 tokens
    (768, 144, 2, 64, 0, 777),       # no low-rank stages; 144 rows in a tile of 256
    (1024, 512, 4, 64, 128, 1030),   # two low-rank stages; last chunk holds 6 tokens
    (2048, 384, 3, 128, 40, 512),    # rank padded inside a stage
    (1024, 256, 4, 128, 16, 40),     # below 512 tokens the two-CTA kernel serves layers with few row tiles:
    (768, 144, 2, 64, 17, 130),      # one accumulator, token boxes that reach past the batch,
    (2048, 384, 3, 64, 64, 300),     # two accumulators with a ragged second one
])
def test_large_batches_pair_two_ctas_on_a_tile(n, m, bits, g, r, T):
    """512 tokens and more: the prefill kernel puts the two CTAs of a cluster on one tile of 256 rows x 512 tokens and
    cuts the tiles of the last wave along K (their partial sums are added by a second kernel).  Run with the library's
    choice of K parts, with none, and with 2, 3 and 4; and with one CTA per tile on the same inputs."""
    layer = random_layer_np(n, m, bits, g, r, seed=n + m + T)
    d = lopro.make_desc(n, m, bits, g, 128, identity_cols=128, rank=r)
    x_bits = synth.activations(T, n, seed=T, outlier_frac=0.01)
    with lopro.configured(lopro.OPT_NO_CHUNKS, 1):
        _pair_kernel_cases(layer, d, x_bits, T)


def _pair_kernel_cases(layer, d, x_bits, T):
    assert lopro.linear_fwd_path(d, T)[0] == lopro.PATH_PREFILL
    launches = set()
    for parts in (-1, 0, 2, 3, 4):
        with lopro.configured(lopro.OPT_PREFILL_PAIRS, parts):
            launches.add(lopro.linear_fwd_path(d, T)[1])
            _check_forward_once(layer, d, x_bits, None, GATE_A, GATE_B)
    assert len(launches) == 2                       # with and without the kernel that adds the K parts
    blob = _pack(layer, d)
    x = bf16_bits_to_device(x_bits)
    y_pair = lopro.linear_fwd(d, blob, x, lopro.OUT_F32)
    with lopro.configured(lopro.OPT_NO_CTA_PAIRS, 1):
        _check_forward_once(layer, d, x_bits, None, GATE_A, GATE_B)
        y_single = lopro.linear_fwd(d, blob, x, lopro.OUT_F32)
    # the same products summed in the same K order by both kernels
    scale = y_single.abs().max().item()
    assert (y_pair - y_single).abs().max().item() <= 1e-5 * scale


@pytest.mark.parametrize("bits,g", [(4, 128), (3, 64), (2, 64)])
@pytest.mark.parametrize("T", [1, 2, 5, 8])
@pytest.mark.parametrize("n,m,r,b", [(2048, 144, 17, 128), (4096, 528, 32, 256), (4096, 64, 0, 64)])
def test_small_batch_path_row_and_token_edges(bits, g, T, n, m, r, b):
    # small-batch path with row counts that leave the last CTA half empty (m % 32 = 16) and few rows overall
    layer = random_layer_np(n, m, bits, g, r, seed=n + m + bits + T)
    d = lopro.make_desc(n, m, bits, g, b, identity_cols=b, rank=r)
    _check_forward(layer, d, synth.activations(T, n, seed=T + 3, outlier_frac=0.01))


@pytest.mark.parametrize("r", [40, 64, 128, 256])
@pytest.mark.parametrize("T", [3, 8])
def test_prologue_row_ctas_for_one_two_four_and_eight_tokens(r, T):
    # the prologue gives a row CTA of t = B x 1, 2, 4 or 8 tokens depending on the padded rank (48, 64, 128, 256 here)
    n, m, bits, g = 2304, 80, 4, 128                          # 36 steps: a ragged third stage; 80 rows: half-empty CTA
    d = lopro.make_desc(n, m, bits, g, 128, identity_cols=128, rank=r)
    assert lopro.linear_fwd_path(d, T)[0] == lopro.PATH_WIDE
    layer = random_layer_np(n, m, bits, g, r, seed=r + T)
    _check_forward(layer, d, synth.activations(T, n, seed=r, outlier_frac=0.01))


def _tall_rows(tiles_per_sm, extra_tiles):
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    return 16 * (sms * tiles_per_sm + extra_tiles)


@pytest.mark.parametrize("bits,g,r", [(4, 128, 32), (3, 64, 17), (2, 64, 128), (4, 256, 0)])
@pytest.mark.parametrize("T", [1, 8, 16, 32])
@pytest.mark.parametrize("per_sm,extra", [(2, 1), (4, 100), (5, 7), (6, 3)])
def test_tall_layers_persistent_kernel(bits, g, r, T, per_sm, extra):
    # more 16-row tiles than twice the SM count: the persistent kernel, with runs of tiles per CTA that end in
    # groups of 1, 2 and 3 tiles (2/3, 4/4+1, 4+1/4+2, 4+2/4+3 tiles per CTA) and a ragged last stage (36 steps)
    n, m = 2304, _tall_rows(per_sm, extra)
    d = lopro.make_desc(n, m, bits, g, 64, identity_cols=64, rank=r)
    assert lopro.linear_fwd_path(d, T)[0] == lopro.PATH_TALL
    layer = random_layer_np(n, m, bits, g, r, seed=m + bits + T)
    _check_forward(layer, d, synth.activations(T, n, seed=T + 11, outlier_frac=0.01))


@pytest.mark.parametrize("g", [1024, 2048, 4096])
@pytest.mark.parametrize("T,m", [(8, 160), (16, 160), (8, None)])
def test_groups_as_long_as_or_longer_than_a_stage(g, T, m):
    # a stage of the small-batch kernels holds 1024 columns: groups of exactly one stage, of two stages and of
    # the whole row (one scale per row), on the 32-warp, the 16-warp and the persistent kernel
    n = 4096
    m = _tall_rows(2, 5) if m is None else m
    d = lopro.make_desc(n, m, 4, g, 128, identity_cols=128, rank=16)
    want = {(8, False): lopro.PATH_WIDE, (16, False): lopro.PATH_STREAM, (8, True): lopro.PATH_TALL}[(T, m > 160)]
    assert lopro.linear_fwd_path(d, T)[0] == want
    layer = random_layer_np(n, m, 4, g, 16, seed=g + T)
    _check_forward(layer, d, synth.activations(T, n, seed=T + g))


@pytest.mark.parametrize("T,n,m,path", [(33, 1024, 4096, "tall"), (96, 1024, 4096, "tall"), (128, 1024, 4096, "prefill"),
                                        (64, 1024, 11008, "tall"), (65, 1024, 11008, "prefill"),
                                        (64, 4096, 4096, "tall"), (65, 4096, 4096, "prefill"),
                                        (40, 2048, 2048, "stream")])
def test_token_counts_above_32_run_as_chunks_where_that_is_estimated_faster(T, n, m, path):
    # one prologue, then chunks of 32 tokens through the small-batch kernels (a ragged last chunk) while
    # chunks x (3 + 0.45e-6 m n) us stays below the estimate for the tensor-core kernels (per 64-column stage and wave)
    d = lopro.make_desc(n, m, 4, 128, 128, identity_cols=128, rank=16)
    got, launches = lopro.linear_fwd_path(d, T)
    assert lopro.PATH_NAMES[got] == path
    if path != "prefill":
        assert launches == 1 + (T + 31) // 32
    layer = random_layer_np(n, m, 4, 128, 16, seed=T + m)
    rows = None if n * m <= 1 << 22 else np.arange(0, m, 7)
    _check_forward(layer, d, synth.activations(T, n, seed=T + 1), rows=rows)


def test_rotated_entry_on_a_bf16_rounding_boundary():
    # 128 tokens drawn with seed 128: one rotated outlier entry lies within fp32 rounding distance of the midpoint of
    # two bf16 values; the fp32 butterflies of the kernel and the fp64 oracle may round it to different sides (inside
    # the rotation's own tolerance), which alone moves one output of that token past 1e-3.  Gate B then holds
    # against the mirrored oracle evaluated for either side (_gate_b_with_ties).
    T, n, m = 128, 1024, 4096
    d = lopro.make_desc(n, m, 4, 128, 128, identity_cols=128, rank=16)
    layer = random_layer_np(n, m, 4, 128, 16, seed=T + m)
    _check_forward(layer, d, synth.activations(T, n, seed=T))


def test_tall_kernel_agrees_with_the_per_group_kernel():
    # both small-batch kernels sum the same products in fp32 in different orders: outputs agree to fp32 rounding
    n, m, bits, g, r, T = 1024, _tall_rows(4, 9), 4, 128, 32, 8
    d = lopro.make_desc(n, m, bits, g, 128, rank=r)
    layer = random_layer_np(n, m, bits, g, r, seed=3)
    blob = _pack(layer, d)
    x = bf16_bits_to_device(synth.activations(T, n, seed=4))
    y_tall = lopro.linear_fwd(d, blob, x, lopro.OUT_F32)
    with lopro.configured(lopro.OPT_NO_TALL, 1):
        assert lopro.linear_fwd_path(d, T)[0] in (lopro.PATH_STREAM, lopro.PATH_WIDE)
        y_stream = lopro.linear_fwd(d, blob, x, lopro.OUT_F32)
    torch.cuda.synchronize()
    scale = y_stream.abs().max().item()
    assert (y_tall - y_stream).abs().max().item() <= 1e-5 * scale


def test_outputs_can_be_strided_and_calls_repeat_bitwise():
    n, m, bits, g, r, T = 1024, 256, 4, 128, 16, 8
    layer = random_layer_np(n, m, bits, g, r, seed=1)
    d = lopro.make_desc(n, m, bits, g, 128, rank=r)
    blob = _pack(layer, d)
    x = bf16_bits_to_device(synth.activations(T, n, seed=2))
    y1 = lopro.linear_fwd(d, blob, x)
    ybuf = torch.zeros((T, m + 32), dtype=torch.bfloat16, device="cuda")
    lopro.linear_fwd(d, blob, x, y=ybuf[:, :m])
    y2 = lopro.linear_fwd(d, blob, x)
    assert torch.equal(y1, ybuf[:, :m]) and torch.equal(y1, y2)     # split-K order is fixed
    assert torch.count_nonzero(ybuf[:, m:]) == 0


@pytest.mark.parametrize("T,pad", [(8, 3), (16, 5), (40, 3), (300, 8), (300, 1)])
def test_strided_outputs_on_every_path(T, pad):
    # y with a row stride that is not the row length: odd strides take the scalar stores of the prefill epilogue,
    # strides that are multiples of 8 its 16-byte stores; the columns beyond m must stay untouched
    n, m, bits, g, r = 1024, 16 * (2 * torch.cuda.get_device_properties(0).multi_processor_count + 3) if T == 16 else 400, 4, 128, 16
    d = lopro.make_desc(n, m, bits, g, 128, rank=r)
    layer = random_layer_np(n, m, bits, g, r, seed=T + pad)
    blob = _pack(layer, d)
    x = bf16_bits_to_device(synth.activations(T, n, seed=pad))
    y_ref = lopro.linear_fwd(d, blob, x)
    ybuf = torch.full((T, m + pad), 7.0, dtype=torch.bfloat16, device="cuda")
    lopro.linear_fwd(d, blob, x, y=ybuf[:, :m])
    torch.cuda.synchronize()
    assert torch.equal(ybuf[:, :m], y_ref)
    assert torch.all(ybuf[:, m:] == 7.0)


def test_forward_argument_errors():
    n, m = 512, 64
    layer = random_layer_np(n, m, 4, 128, 0, seed=1)
    d = lopro.make_desc(n, m, 4, 128, 64, rank=0)
    blob = _pack(layer, d)
    x = torch.zeros((4, n), dtype=torch.bfloat16, device="cuda")
    small = torch.zeros(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(lopro.LoproError) as e:
        lopro.linear_fwd(d, blob, x, workspace=small)
    assert e.value.status == lopro.ERR_BUFFER_TOO_SMALL
    y = lopro.linear_fwd(d, blob, x[:0])                        # T = 0
    assert y.shape == (0, m)


@pytest.mark.parametrize("T", [8, 40, 300])  # small batch, chunks of 32 tokens, tensor-core path
def test_host_entry_point_matches_device_entry_point(T):
    n, m, bits, g, r = 1024, 256, 4, 128, 16
    layer = random_layer_np(n, m, bits, g, r, seed=4)
    d = lopro.make_desc(n, m, bits, g, 128, rank=r)
    blob = _pack(layer, d)
    x_bits = synth.activations(T, n, seed=5)
    x = bf16_bits_to_device(x_bits)
    y_dev = lopro.linear_fwd(d, blob, x)
    xh = torch.from_numpy(x_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    yh = torch.empty((T, m), dtype=torch.bfloat16).pin_memory()
    ws = torch.zeros(lopro.workspace_bytes(d, T) + lopro.host_staging_bytes(d, T), dtype=torch.uint8, device="cuda")
    lopro.linear_fwd_host(d, blob, xh, yh, ws)
    torch.cuda.synchronize()
    assert torch.equal(yh, y_dev.cpu())


def test_a_bounded_wait_that_runs_out_reports_a_timeout():
    # the library's own self-test: a barrier that nothing completes, waited on with the bounded wait every
    # forward kernel uses; the wait gives up, the kernel returns normally and the status word says so
    word = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    lopro.selftest_wait(word)
    torch.cuda.synchronize()
    assert int(word.item()) == lopro.ERR_TIMEOUT
    # the context is intact: an ordinary forward still runs and reports OK
    n, m = 512, 64
    d = lopro.make_desc(n, m, 4, 128, 64, rank=0)
    blob = _pack(random_layer_np(n, m, 4, 128, 0, seed=1), d)
    ws = torch.zeros(lopro.workspace_bytes(d, 4), dtype=torch.uint8, device="cuda")
    y = lopro.linear_fwd(d, blob, torch.ones((4, n), dtype=torch.bfloat16, device="cuda"), workspace=ws)
    torch.cuda.synchronize()
    assert lopro.workspace_status(ws) == lopro.OK and torch.isfinite(y.float()).all()


@pytest.mark.parametrize("n,m,bits,g,r,T", [
    (4096, 4096, 4, 128, 32, 1), (4096, 4096, 4, 128, 32, 8), (2048, 272, 3, 64, 17, 32),     # small-batch kernels
    (2048, 5008, 2, 64, 128, 16),                                                              # persistent kernel
    (1024, 256, 4, 128, 16, 40), (1024, 4096, 4, 128, 16, 100),                               # chunks / tensor-core kernels
    (1024, 512, 4, 64, 128, 300), (2048, 384, 3, 128, 40, 777),                               # K parts in the workspace
])
def test_nothing_is_written_outside_the_workspace_or_the_output(n, m, bits, g, r, T):
    """Guard bytes behind the workspace (sized exactly by lopro_workspace_bytes) and behind every output row (ldy > m)
    keep their pattern on every path; so does the packed layer (a forward only reads it)."""
    layer = random_layer_np(n, m, bits, g, r, seed=n + T)
    d = lopro.make_desc(n, m, bits, g, 128, identity_cols=128, rank=r)
    blob = _pack(layer, d)
    blob_before = blob.clone()
    x = bf16_bits_to_device(synth.activations(T, n, seed=T))
    need, guard, pad = lopro.workspace_bytes(d, T), 1 << 16, 24
    for no_chunks in (0, 1):
        with lopro.configured(lopro.OPT_NO_CHUNKS, no_chunks):
            for out_dtype, tdt in ((lopro.OUT_BF16, torch.bfloat16), (lopro.OUT_F32, torch.float32)):
                buf = torch.full((need + guard,), 0xA5, dtype=torch.uint8, device="cuda")
                y = torch.full((T, m + pad), -7.0, dtype=tdt, device="cuda")
                lopro.linear_fwd(d, blob, x, out_dtype, workspace=buf[:need], y=y[:, :m])
                torch.cuda.synchronize()
                assert lopro.workspace_status(buf) == lopro.OK
                assert bool((buf[need:] == 0xA5).all())
                assert bool((y[:, m:] == -7.0).all()) and bool(torch.isfinite(y[:, :m].float()).all())
    assert torch.equal(blob, blob_before)
