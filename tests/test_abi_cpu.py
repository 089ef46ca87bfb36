"""Host-only checks of the C ABI: the library loads without a GPU, exports every symbol the header
declares, validates descriptors, and sizes the blob by the storage accounting of Eq. 13."""
import os
import re

import pytest

from oracle import lopro_oracle as o
from paper_2601_19675_b200 import build, lopro

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "lopro.h")).read() + open(os.path.join(ROOT, "include", "lopro_block.h")).read() + \
        open(os.path.join(ROOT, "include", "lopro_vq.h")).read()
    return sorted(set(re.findall(r"LOPRO_API[^;(]*?\b(lopro_\w+)\s*\(", text)))


def test_header_declares_what_binding_lists():
    assert _declared_symbols() == sorted(lopro.SYMBOLS)


def test_library_exports_every_declared_symbol():
    L = lopro.lib()
    for name in _declared_symbols():
        assert hasattr(L, name), name
    assert lopro.version() >= 100
    assert lopro.status_str(lopro.OK) == "ok"
    assert "timed out" in lopro.status_str(lopro.ERR_TIMEOUT)


@pytest.mark.parametrize("kw,expect", [
    (dict(), lopro.OK),
    (dict(bits=5), lopro.ERR_INVALID_ARG),
    (dict(bits=1), lopro.ERR_INVALID_ARG),
    (dict(block_size=96), lopro.ERR_INVALID_ARG),          # b_H must be a power of two (Eq. 6)
    (dict(block_size=2048), lopro.ERR_INVALID_ARG),
    (dict(identity_cols=100), lopro.ERR_INVALID_ARG),      # (n - b_I) must be a whole number of blocks
    (dict(identity_cols=0), lopro.OK),
    (dict(identity_cols=4096), lopro.OK),                  # rotation disabled
    (dict(group_size=100), lopro.ERR_INVALID_ARG),         # g must divide n
    (dict(group_size=32), lopro.ERR_UNSUPPORTED),
    (dict(d_in=4096 + 32, identity_cols=32 + 128), lopro.ERR_INVALID_ARG),
    (dict(d_out=4100), lopro.ERR_UNSUPPORTED),
    (dict(rank=-1), lopro.ERR_INVALID_ARG),
    (dict(rank=17), lopro.OK),
    (dict(layout=7), lopro.ERR_INVALID_ARG),
])
def test_descriptor_domain(kw, expect):
    base = dict(d_in=4096, d_out=4096, bits=4, group_size=128, block_size=128, identity_cols=128, rank=32)
    base.update(kw)
    d = lopro.make_desc(**base)
    assert lopro.check_desc(d) == expect
    assert (lopro.packed_bytes(d) > 0) == (expect == lopro.OK)


@pytest.mark.parametrize("m,n,bits,g,r", [(4096, 4096, 4, 128, 32), (11008, 4096, 3, 64, 64), (28672, 8192, 2, 64, 128),
                                          (512, 512, 4, 128, 16)])
def test_blob_size_follows_eq13_accounting(m, n, bits, g, r):
    # Eq. 13 with this library's widths: d_q bits per code, 16-bit scale and 16-bit zero per group,
    # 16-bit factor entries (rank padded to 16), 32-bit permutation entries; plus a 256-byte header
    # and at most 255 bytes of padding after each of the eight sections.
    d = lopro.make_desc(n, m, bits, g, 64, rank=r)
    r_pad = (r + 15) // 16 * 16
    payload_bits = m * n * (o.average_bits(m, n, bits, 32, g, r_pad, 16) - 2 * 32 / n - r_pad * 32 / (m * n)) + 32 * n
    nbytes = lopro.packed_bytes(d)
    assert payload_bits / 8 + 256 <= nbytes <= payload_bits / 8 + 256 + 8 * 256
    total = 0
    for sec in range(8):
        off, sz = lopro.packed_section(d, sec)
        assert off % 256 == 0 and off >= total
        total = off + sz
    assert total <= nbytes


def test_workspace_size_is_monotone_in_tokens():
    d = lopro.make_desc(4096, 4096, 4, 128, 128, rank=32)
    sizes = [lopro.workspace_bytes(d, t) for t in (0, 1, 7, 8, 9, 32, 33, 2048)]
    assert all(a <= b for a, b in zip(sizes, sizes[1:])) and sizes[0] > 0
    # every token count, on the shapes of the configurations (the prefill tiling's last wave shrinks and grows with T)
    for n, m, bits, g, b, r in ((4096, 11008, 3, 64, 128, 64), (8192, 28672, 2, 64, 256, 128), (4096, 4096, 4, 128, 128, 32),
                                (32768, 1024, 4, 128, 256, 256), (4096, 4096, 4, 128, 128, 0), (8192, 8192, 2, 64, 256, 17)):
        dd = lopro.make_desc(n, m, bits, g, b, identity_cols=b, rank=r)
        assert lopro.workspace_bytes(dd, 1) > 0
        prev = 0
        for t in range(0, 8193):
            cur = lopro.workspace_bytes(dd, t)
            assert cur >= prev, (n, m, t)
            prev = cur
    assert lopro.workspace_bytes(d, -1) == 0
    assert lopro.host_staging_bytes(d, 8) >= 8 * 4096 * 2 * 2


def test_forward_path_query_names_the_small_batch_and_general_paths():
    d = lopro.make_desc(4096, 4096, 4, 128, 128, rank=32)
    assert lopro.linear_fwd_path(d, 8) == (lopro.PATH_WIDE, 2)         # prologue + streaming kernel, 32-warp variant
    assert lopro.linear_fwd_path(d, 16) == (lopro.PATH_STREAM, 2)      # prologue + streaming kernel
    assert lopro.linear_fwd_path(d, 0) == (0, 0) and lopro.linear_fwd_path(d, -3) == (0, 0)
    wide = lopro.make_desc(4096, 4096, 4, 128, 1024, identity_cols=0, rank=32)  # b_H beyond the prologue's 256
    path, launches = lopro.linear_fwd_path(wide, 8)
    assert path == lopro.PATH_GENERAL and launches == 3                # rotation, B x, product
    assert lopro.linear_fwd_path(lopro.make_desc(4096, 4096, 4, 128, 1024, identity_cols=0, rank=0), 8)[1] == 2
    bad = lopro.make_desc(4096, 4096, 5, 128, 128, rank=32)
    assert lopro.linear_fwd_path(bad, 8)[0] == 0


def test_null_and_bad_arguments_are_rejected_before_any_cuda_call():
    import ctypes
    L = lopro.lib()
    d = lopro.make_desc(512, 512, 4, 128, 64, rank=16)
    assert L.lopro_pack(None, None, None, None, None, None, None, None, 0, None) == lopro.ERR_INVALID_ARG
    assert L.lopro_pack(ctypes.byref(d), None, None, None, None, None, None, None, 0, None) == lopro.ERR_INVALID_ARG
    assert L.lopro_rotate(ctypes.byref(d), None, None, 512, None, 512, 4, None) == lopro.ERR_INVALID_ARG
    assert L.lopro_rotate(ctypes.byref(d), None, None, 512, None, 512, 0, None) == lopro.OK      # T = 0: no-op
    assert L.lopro_rotate(ctypes.byref(d), None, None, 512, None, 512, -1, None) == lopro.ERR_INVALID_ARG
    assert L.lopro_linear_fwd(ctypes.byref(d), None, None, 512, None, 512, 0, 0, None, 0, None) == lopro.OK
    assert L.lopro_linear_fwd(ctypes.byref(d), None, None, 512, None, 512, 0, 4, None, 0, None) == lopro.ERR_INVALID_ARG
    assert L.lopro_linear_fwd(ctypes.byref(d), None, None, 512, None, 512, 9, 4, None, 0, None) == lopro.ERR_INVALID_ARG
    dc = lopro.make_desc(512, 512, 4, 128, 64, rank=16, layout=lopro.LAYOUT_CANONICAL)
    assert L.lopro_linear_fwd(ctypes.byref(dc), None, None, 512, None, 512, 0, 4, None, 0, None) == lopro.ERR_UNSUPPORTED
    # misaligned pointers and short leading dimensions (fake non-null addresses are never dereferenced)
    fake = ctypes.c_void_p(0x1000)
    odd = ctypes.c_void_p(0x1002)
    assert L.lopro_rotate(ctypes.byref(d), fake, odd, 512, fake, 512, 4, None) == lopro.ERR_INVALID_ARG
    assert L.lopro_rotate(ctypes.byref(d), fake, fake, 500, fake, 512, 4, None) == lopro.ERR_INVALID_ARG
    assert L.lopro_linear_fwd(ctypes.byref(d), fake, fake, 512, fake, 100, 0, 4, fake, 1 << 30, None) == lopro.ERR_INVALID_ARG
    assert L.lopro_linear_fwd(ctypes.byref(d), fake, fake, 512, fake, 512, 0, 4, fake, 16, None) == lopro.ERR_BUFFER_TOO_SMALL


@pytest.mark.parametrize("n,r", [(4096, 32), (8192, 128), (32768, 17), (4096, 0)])
def test_workspace_size_never_decreases_with_the_token_count(n, r):
    # a workspace sized once for the largest batch must serve every smaller one
    d = lopro.make_desc(n, 256, 2, 64, 256, rank=r)
    prev = 0
    for t in range(1, 8193):
        cur = lopro.workspace_bytes(d, t)
        assert cur >= prev, (t, cur, prev)
        prev = cur


def test_configure_rejects_unknown_options():
    import ctypes
    L = lopro.lib()
    assert L.lopro_configure(99, 1) == lopro.ERR_INVALID_ARG
    assert L.lopro_configure(-1, 1) == lopro.ERR_INVALID_ARG
    d = lopro.make_desc(4096, 4096, 4, 128, 128, rank=32)
    with lopro.configured(lopro.OPT_NO_WIDE, 1):
        assert lopro.linear_fwd_path(d, 8) == (lopro.PATH_STREAM, 2)
    assert lopro.linear_fwd_path(d, 8) == (lopro.PATH_WIDE, 2)
    assert L.lopro_selftest_wait(None, None) == lopro.ERR_INVALID_ARG
    assert L.lopro_selftest_wait(ctypes.c_void_p(0x1002), None) == lopro.ERR_INVALID_ARG


def test_fp8_lowrank_record_reproduces_the_printed_storage_overhead(golden_dir):
    # Appendix A.2 / rank-ablation table: U and V in fp8 (d_r = 8) at r = 16 cost about 0.05 bit per weight over the
    # linears of a 7B model and 0.04 over a 13B model; the blob's A and B sections of the FP8 format hold exactly that
    gold = {}
    with open(os.path.join(golden_dir, "avg_bits.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v, tol, _ = line.split()
                gold[k] = (float(v), float(tol))
    shapes = {"7b": [(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)],
              "13b": [(5120, 5120)] * 4 + [(13824, 5120)] * 2 + [(5120, 13824)]}
    for model, sh in shapes.items():
        bits = weights = 0
        for m, n in sh:
            d = lopro.make_desc(n, m, 4, 128, 128, rank=16, lowrank_format=lopro.LOWRANK_FP8)
            assert lopro.check_desc(d) == lopro.OK
            bits += 8 * (lopro.packed_section(d, lopro.SEC_A)[1] + lopro.packed_section(d, lopro.SEC_B)[1])
            weights += m * n
            # Sigma and s: 16 bits per entry, as Eq. 13 counts them (r d_o and n d_o)
            assert lopro.packed_section(d, lopro.SEC_SIGMA)[1] == 16 * 2 and lopro.packed_section(d, lopro.SEC_S)[1] == n * 2
        val, tol = gold[f"rbit_{model}_r16"]
        assert abs(bits / weights - val) <= tol
    # the folded fp16 format has no such sections and twice the factor bytes
    d16 = lopro.make_desc(4096, 4096, 4, 128, 128, rank=16)
    d8 = lopro.make_desc(4096, 4096, 4, 128, 128, rank=16, lowrank_format=lopro.LOWRANK_FP8)
    assert lopro.packed_section(d16, lopro.SEC_SIGMA)[1] == 0 and lopro.packed_section(d16, lopro.SEC_S)[1] == 0
    assert lopro.packed_section(d16, lopro.SEC_A)[1] == 2 * lopro.packed_section(d8, lopro.SEC_A)[1]
    assert lopro.check_desc(lopro.make_desc(4096, 4096, 4, 128, 128, rank=0, lowrank_format=lopro.LOWRANK_FP8)) == lopro.ERR_INVALID_ARG
    assert lopro.check_desc(lopro.make_desc(4096, 4096, 4, 128, 128, rank=16, lowrank_format=3)) == lopro.ERR_INVALID_ARG


def test_offline_side_workspace_sizes():
    # the layer quantizer keeps a copy of W (deflated in place by the rank-1 sketch) besides its small vectors
    d = lopro.make_desc(4096, 11008, 4, 128, 128, rank=16)
    need = lopro.quantize_workspace_bytes(d)
    assert need >= 4096 * 11008 * 4 and need <= 4096 * 11008 * 4 * 1.1
    assert lopro.lib().lopro_r1svd_workspace_bytes(11008, 4096) >= (11008 // 32) * 4096 * 4
    # rank 0: no copy, no sketch workspace
    assert lopro.quantize_workspace_bytes(lopro.make_desc(4096, 4096, 2, 64, 256, rank=0)) < 1 << 20
    # rows longer than two fp32 copies in one CTA's shared memory are refused
    assert lopro.quantize_workspace_bytes(lopro.make_desc(32768, 64, 4, 128, 128, rank=0)) == 0
    assert lopro.lib().lopro_r1svd_workspace_bytes(0, 16) == 0
