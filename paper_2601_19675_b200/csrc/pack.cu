// Layout transforms between plain arrays and the packed blob, and the input checks of lopro_pack.
// One-time set-up work: written for clarity, not speed.
#include "common.cuh"

namespace lopro {

namespace {

__device__ __forceinline__ bool f16_is_finite(uint16_t h) { return (h & 0x7C00u) != 0x7C00u; }

__global__ void validate_kernel(const uint8_t* __restrict__ codes, const uint16_t* __restrict__ scales,
                                const uint16_t* __restrict__ zeros, const int32_t* __restrict__ perm,
                                int* __restrict__ marks, uint32_t* __restrict__ invalid, size_t n_codes,
                                size_t n_groups_total, int n, int bits) {
    const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    uint32_t bad = 0;
    for (size_t i = tid; i < n_codes; i += stride)
        if (codes[i] >> bits) bad |= kInvalidCode;
    for (size_t i = tid; i < n_groups_total; i += stride) {
        const uint16_t s = scales[i], z = zeros[i];
        if (!f16_is_finite(s) || (s & 0x7FFFu) == 0) bad |= kInvalidScale;
        if (!f16_is_finite(z)) bad |= kInvalidZero;
    }
    for (size_t i = tid; i < (size_t)n; i += stride) {
        const int p = perm[i];
        if (p < 0 || p >= n) {
            bad |= kInvalidPermRange;
        } else if (atomicExch(&marks[p], 1) != 0) {
            bad |= kInvalidPermDuplicate;
        }
    }
    if (bad) atomicOr(invalid, bad);
}

__device__ __forceinline__ uint32_t load_code(const uint8_t* __restrict__ codes, int n, int bits, int row, int k) {
    return (uint32_t)codes[(size_t)row * n + k] & ((1u << bits) - 1u);
}

// Canonical bit stream: one thread per output word.
__global__ void pack_canonical_kernel(const uint8_t* __restrict__ codes, uint32_t* __restrict__ words, int m, int n,
                                      int bits) {
    const int wpr = n * bits / 32;
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)m * wpr) return;
    const int row = (int)(idx / wpr), w = (int)(idx % wpr);
    const int bit0 = 32 * w;
    uint32_t out = 0;
    for (int k = bit0 / bits; k * bits < bit0 + 32 && k < n; ++k) {
        const uint32_t c = load_code(codes, n, bits, row, k);
        const int pos = k * bits - bit0;  // may be negative: code straddles the previous word
        out |= pos >= 0 ? (c << pos) : (c >> (-pos));
    }
    words[idx] = out;
}

// Fragment layout: one thread per (16-row tile, 64-column step, lane); writes `bits` words.
__global__ void pack_fragment_kernel(const uint8_t* __restrict__ codes, uint32_t* __restrict__ words, int m, int n,
                                     int bits) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t total = (size_t)(m / 16) * (n / 64) * 32;
    if (idx >= total) return;
    const int lane = (int)(idx & 31);
    const size_t tile = idx >> 5;
    const int ks = (int)(tile % (n / 64)), rt = (int)(tile / (n / 64));
    const int gq = lane >> 2, tg = lane & 3;
    uint32_t w[4] = {0, 0, 0, 0};
    for (int pi = 0; pi < 16; ++pi) {
        const int j = pi >> 2, rho = pi & 3;
        const int row = rt * 16 + gq + 8 * (rho & 1);
        const int k = ks * 64 + 16 * j + 8 * (rho >> 1) + 2 * tg;
        const uint32_t lo = load_code(codes, n, bits, row, k), hi = load_code(codes, n, bits, row, k + 1);
        if (bits == 4) {
            w[j] |= (lo << (4 * rho)) | (hi << (16 + 4 * rho));
        } else if (bits == 2) {
            w[pi >> 3] |= (lo << (2 * (pi & 7))) | (hi << (16 + 2 * (pi & 7)));
        } else if (pi < 15) {
            w[pi / 5] |= (lo << (3 * (pi % 5))) | (hi << (16 + 3 * (pi % 5)));
        } else {
            for (int b = 0; b < 3; ++b) w[b] |= (((lo >> b) & 1u) << 15) | (((hi >> b) & 1u) << 31);
        }
    }
    for (int b = 0; b < bits; ++b) words[idx * bits + b] = w[b];
}

// Row-block layout: one thread per (row, 64-column step); writes the row's 2 q words of the step.
__global__ void pack_rowblock_kernel(const uint8_t* __restrict__ codes, uint32_t* __restrict__ words, int m, int n,
                                     int bits) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int nsteps = n / 64;
    if (idx >= (size_t)m * nsteps) return;
    const int row = (int)(idx / nsteps), ks = (int)(idx % nsteps);
    const int rb = row >> 7, r = row & 127, R = rb_rows(m, rb);
    uint32_t* dst = words + rb_step_word(bits, nsteps, m, rb, ks);
    for (int hs = 0; hs < 2; ++hs) {
        uint32_t w[4] = {0, 0, 0, 0};
        for (int pi = 0; pi < 16; ++pi) {
            const int k = ks * 64 + hs * 32 + 2 * pi;
            const uint32_t lo = load_code(codes, n, bits, row, k), hi = load_code(codes, n, bits, row, k + 1);
            if (bits == 4) {
                w[pi >> 2] |= (lo << (4 * (pi & 3))) | (hi << (16 + 4 * (pi & 3)));
            } else if (bits == 2) {
                w[pi >> 3] |= (lo << (2 * (pi & 7))) | (hi << (16 + 2 * (pi & 7)));
            } else if (pi < 15) {
                w[pi / 5] |= (lo << (3 * (pi % 5))) | (hi << (16 + 3 * (pi % 5)));
            } else {
                for (int b = 0; b < 3; ++b) w[b] |= (((lo >> b) & 1u) << 15) | (((hi >> b) & 1u) << 31);
            }
        }
        for (int b = 0; b < bits; ++b) dst[rb_word_in_step(bits, R, r, hs * bits + b)] = w[b];
    }
}

__device__ __forceinline__ uint32_t read_code(const uint32_t* __restrict__ words, int layout, int bits, int m, int n,
                                              int row, int k) {
    if (layout == LOPRO_LAYOUT_ROWBLOCK) {
        const FragPos p = rb_pos(bits, n, m, row, k);
        if (!p.scattered) return (words[p.word] >> p.shift) & ((1u << bits) - 1u);
        uint32_t c = 0;
        for (int b = 0; b < 3; ++b) c |= ((words[rb_halfstep_word(bits, n, m, row, k, b)] >> p.shift) & 1u) << b;
        return c;
    }
    if (layout == LOPRO_LAYOUT_FRAGMENT) {
        const FragPos p = frag_pos(bits, n, row, k);
        if (!p.scattered) return (words[p.word] >> p.shift) & ((1u << bits) - 1u);
        uint32_t c = 0;
        for (int b = 0; b < 3; ++b) c |= ((words[p.word + b] >> p.shift) & 1u) << b;
        return c;
    }
    const size_t bit = (size_t)row * n * bits + (size_t)k * bits;
    const size_t w = bit >> 5;
    const int sh = (int)(bit & 31);
    uint32_t c = words[w] >> sh;
    if (sh + bits > 32) c |= words[w + 1] << (32 - sh);
    return c & ((1u << bits) - 1u);
}

__global__ void unpack_codes_kernel(const uint32_t* __restrict__ words, uint8_t* __restrict__ codes, int m, int n,
                                    int bits, int layout) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)m * n) return;
    codes[idx] = (uint8_t)read_code(words, layout, bits, m, n, (int)(idx / n), (int)(idx % n));
}

__global__ void unpack_words_kernel(const uint32_t* __restrict__ words, uint32_t* __restrict__ out, int m, int n,
                                    int bits, int layout) {
    const int wpr = n * bits / 32;
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)m * wpr) return;
    const int row = (int)(idx / wpr), w = (int)(idx % wpr);
    const int bit0 = 32 * w;
    uint32_t o = 0;
    for (int k = bit0 / bits; k * bits < bit0 + 32 && k < n; ++k) {
        const uint32_t c = read_code(words, layout, bits, m, n, row, k);
        const int pos = k * bits - bit0;
        o |= pos >= 0 ? (c << pos) : (c >> (-pos));
    }
    out[idx] = o;
}

// (scale, zero) pairs.  to_blob: plain [m][ng] arrays -> blob order; else the reverse.
__global__ void scalezero_kernel(uint16_t* __restrict__ scales, uint16_t* __restrict__ zeros,
                                 uint32_t* __restrict__ sz, int m, int ng, int layout, bool to_blob) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)m * ng) return;
    const int row = (int)(idx / ng), grp = (int)(idx % ng);
    const size_t pos = layout == LOPRO_LAYOUT_FRAGMENT ? sz_frag_index(ng, row, grp)
                       : layout == LOPRO_LAYOUT_ROWBLOCK ? sz_rb_index(ng, m, row, grp) : idx;
    if (to_blob) {
        sz[pos] = (uint32_t)scales[idx] | ((uint32_t)zeros[idx] << 16);
    } else {
        const uint32_t v = sz[pos];
        if (scales) scales[idx] = (uint16_t)(v & 0xFFFFu);
        if (zeros) zeros[idx] = (uint16_t)(v >> 16);
    }
}

// Factor matrices with the rank padded to r_pad (zeros): A [m][r] <-> [m][r_pad], B [r][n] <-> [r_pad][n].
__global__ void copy_padded_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, size_t rows,
                                   int cols, int src_ld, int dst_ld) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * (size_t)cols) return;
    const size_t r = idx / cols;
    const int c = (int)(idx % cols);
    dst[r * dst_ld + c] = src[r * src_ld + c];
}

// byte matrices of the FP8 low-rank record, rank padded with zeros: U [m][r] <-> [m][r_pad], V [r][n] <-> [r_pad][n]
__global__ void copy_padded_bytes_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, size_t rows, int cols,
                                         int src_ld, int dst_ld) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * (size_t)cols) return;
    const size_t r = idx / cols;
    const int c = (int)(idx % cols);
    dst[r * dst_ld + c] = src[r * src_ld + c];
}

// e4m3 has no infinities; S.1111.111 is NaN.  Sigma finite; s finite and non-zero (the forward divides by it).
__global__ void validate_lr8_kernel(const uint8_t* __restrict__ U, size_t n_u, const uint8_t* __restrict__ V, size_t n_v,
                                    const uint16_t* __restrict__ sigma, int r, const uint16_t* __restrict__ svec, int n,
                                    uint32_t* __restrict__ invalid) {
    const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (size_t)gridDim.x * blockDim.x;
    bool bad = false;
    for (size_t i = tid; i < n_u; i += stride) bad |= (U[i] & 0x7Fu) == 0x7Fu;
    for (size_t i = tid; i < n_v; i += stride) bad |= (V[i] & 0x7Fu) == 0x7Fu;
    for (size_t i = tid; i < (size_t)r; i += stride) bad |= !f16_is_finite(sigma[i]);
    for (size_t i = tid; i < (size_t)n; i += stride) bad |= !f16_is_finite(svec[i]) || (svec[i] & 0x7FFFu) == 0;
    if (bad) atomicOr(invalid, kInvalidLowrank);
}

inline unsigned blocks_for(size_t n, int threads) { return (unsigned)((n + threads - 1) / threads); }

}  // namespace

cudaError_t launch_validate(const lopro_desc& d, const uint8_t* codes, const uint16_t* scales, const uint16_t* zeros,
                            const int32_t* perm, void* blob, const BlobLayout& L, cudaStream_t s) {
    // The (not yet written) code section doubles as the mark array of the bijection test:
    // it holds at least m * n / 4 >= 4 n bytes because m >= 16.
    int* marks = (int*)((uint8_t*)blob + L.off[LOPRO_SEC_CODES]);
    uint32_t* invalid = &((BlobHeader*)blob)->invalid;
    const size_t n_codes = (size_t)d.d_out * d.d_in, n_grp = (size_t)d.d_out * (d.d_in / d.group_size);
    validate_kernel<<<1024, 256, 0, s>>>(codes, scales, zeros, perm, marks, invalid, n_codes, n_grp, d.d_in, d.bits);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return cudaMemsetAsync(marks, 0, (size_t)d.d_in * 4, s);
}

cudaError_t launch_pack(const lopro_desc& d, const uint8_t* codes, const uint16_t* scales, const uint16_t* zeros,
                        const int32_t* perm, const uint16_t* A, const uint16_t* B, void* blob, const BlobLayout& L,
                        cudaStream_t s) {
    uint8_t* base = (uint8_t*)blob;
    const int m = d.d_out, n = d.d_in, ng = n / d.group_size;
    uint32_t* words = (uint32_t*)(base + L.off[LOPRO_SEC_CODES]);
    if (d.layout == LOPRO_LAYOUT_FRAGMENT) {
        const size_t total = (size_t)(m / 16) * (n / 64) * 32;
        pack_fragment_kernel<<<blocks_for(total, 256), 256, 0, s>>>(codes, words, m, n, d.bits);
    } else if (d.layout == LOPRO_LAYOUT_ROWBLOCK) {
        const size_t total = (size_t)m * (n / 64);
        pack_rowblock_kernel<<<blocks_for(total, 256), 256, 0, s>>>(codes, words, m, n, d.bits);
    } else {
        const size_t total = (size_t)m * (n * d.bits / 32);
        pack_canonical_kernel<<<blocks_for(total, 256), 256, 0, s>>>(codes, words, m, n, d.bits);
    }
    scalezero_kernel<<<blocks_for((size_t)m * ng, 256), 256, 0, s>>>(
        (uint16_t*)scales, (uint16_t*)zeros, (uint32_t*)(base + L.off[LOPRO_SEC_SCALEZERO]), m, ng, d.layout, true);
    cudaError_t e = cudaMemcpyAsync(base + L.off[LOPRO_SEC_PERM], perm, (size_t)n * 4, cudaMemcpyDeviceToDevice, s);
    if (e != cudaSuccess) return e;
    if (d.rank > 0 && A != nullptr && B != nullptr) {
        copy_padded_kernel<<<blocks_for((size_t)m * d.rank, 256), 256, 0, s>>>(
            A, (uint16_t*)(base + L.off[LOPRO_SEC_A]), (size_t)m, d.rank, d.rank, L.r_pad);
        copy_padded_kernel<<<blocks_for((size_t)d.rank * n, 256), 256, 0, s>>>(
            B, (uint16_t*)(base + L.off[LOPRO_SEC_B]), (size_t)d.rank, n, n, n);
    }
    return cudaGetLastError();
}

cudaError_t launch_pack_lr8(const lopro_desc& d, const uint8_t* U, const uint8_t* V, const uint16_t* sigma, const uint16_t* svec,
                            void* blob, const BlobLayout& L, cudaStream_t s) {
    uint8_t* base = (uint8_t*)blob;
    const int m = d.d_out, n = d.d_in, r = d.rank;
    validate_lr8_kernel<<<256, 256, 0, s>>>(U, (size_t)m * r, V, (size_t)r * n, sigma, r, svec, n, &((BlobHeader*)blob)->invalid);
    copy_padded_bytes_kernel<<<blocks_for((size_t)m * r, 256), 256, 0, s>>>(U, base + L.off[LOPRO_SEC_A], (size_t)m, r, r, L.r_pad);
    copy_padded_bytes_kernel<<<blocks_for((size_t)r * n, 256), 256, 0, s>>>(V, base + L.off[LOPRO_SEC_B], (size_t)r, n, n, n);
    cudaError_t e = cudaMemcpyAsync(base + L.off[LOPRO_SEC_SIGMA], sigma, (size_t)r * 2, cudaMemcpyDeviceToDevice, s);
    if (e != cudaSuccess) return e;
    e = cudaMemcpyAsync(base + L.off[LOPRO_SEC_S], svec, (size_t)n * 2, cudaMemcpyDeviceToDevice, s);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

cudaError_t launch_unpack_lr8(const lopro_desc& d, const void* blob, const BlobLayout& L, uint8_t* U, uint8_t* V,
                              uint16_t* sigma, uint16_t* svec, cudaStream_t s) {
    const uint8_t* base = (const uint8_t*)blob;
    const int m = d.d_out, n = d.d_in, r = d.rank;
    if (U) copy_padded_bytes_kernel<<<blocks_for((size_t)m * r, 256), 256, 0, s>>>(base + L.off[LOPRO_SEC_A], U, (size_t)m, r, L.r_pad, r);
    if (V) copy_padded_bytes_kernel<<<blocks_for((size_t)r * n, 256), 256, 0, s>>>(base + L.off[LOPRO_SEC_B], V, (size_t)r, n, n, n);
    cudaError_t e = cudaSuccess;
    if (sigma) e = cudaMemcpyAsync(sigma, base + L.off[LOPRO_SEC_SIGMA], (size_t)r * 2, cudaMemcpyDeviceToDevice, s);
    if (e != cudaSuccess) return e;
    if (svec) e = cudaMemcpyAsync(svec, base + L.off[LOPRO_SEC_S], (size_t)n * 2, cudaMemcpyDeviceToDevice, s);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

cudaError_t launch_unpack(const lopro_desc& d, const void* blob, const BlobLayout& L, uint8_t* codes, uint32_t* words,
                          uint16_t* scales, uint16_t* zeros, int32_t* perm, uint16_t* A, uint16_t* B,
                          cudaStream_t s) {
    const uint8_t* base = (const uint8_t*)blob;
    const int m = d.d_out, n = d.d_in, ng = n / d.group_size;
    const uint32_t* src = (const uint32_t*)(base + L.off[LOPRO_SEC_CODES]);
    if (codes)
        unpack_codes_kernel<<<blocks_for((size_t)m * n, 256), 256, 0, s>>>(src, codes, m, n, d.bits, d.layout);
    if (words)
        unpack_words_kernel<<<blocks_for((size_t)m * (n * d.bits / 32), 256), 256, 0, s>>>(src, words, m, n, d.bits,
                                                                                          d.layout);
    if (scales || zeros)
        scalezero_kernel<<<blocks_for((size_t)m * ng, 256), 256, 0, s>>>(
            scales, zeros, (uint32_t*)(base + L.off[LOPRO_SEC_SCALEZERO]), m, ng, d.layout, false);
    if (perm) {
        cudaError_t e = cudaMemcpyAsync(perm, base + L.off[LOPRO_SEC_PERM], (size_t)n * 4, cudaMemcpyDeviceToDevice, s);
        if (e != cudaSuccess) return e;
    }
    if (d.rank > 0 && d.lowrank_format == LOPRO_LOWRANK_FOLDED_F16) {
        if (A)
            copy_padded_kernel<<<blocks_for((size_t)m * d.rank, 256), 256, 0, s>>>(
                (const uint16_t*)(base + L.off[LOPRO_SEC_A]), A, (size_t)m, d.rank, L.r_pad, d.rank);
        if (B)
            copy_padded_kernel<<<blocks_for((size_t)d.rank * n, 256), 256, 0, s>>>(
                (const uint16_t*)(base + L.off[LOPRO_SEC_B]), B, (size_t)d.rank, n, n, n);
    }
    return cudaGetLastError();
}

}  // namespace lopro
