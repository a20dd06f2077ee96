// MWQ quantization + packing (Section 3.3.1, Eq. 2 and Eq. 4) and the unpack test hook.
#include "d2moe_common.cuh"

namespace {

constexpr int PACK_THREADS = 256;

__global__ void pack_header_kernel(PackHeader* h, PackLayout L, int n_bits,
                                   int b0, int b1, int b2, int b3, int b4, int b5, int b6, int b7) {
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        h->magic = D2MOE_MAGIC; h->version = D2MOE_LAYOUT_VERSION;
        h->rows = L.rows; h->cols = L.cols; h->g = L.g; h->n_bits = n_bits;
        int b[8] = {b0, b1, b2, b3, b4, b5, b6, b7};
        for (int i = 0; i < 8; ++i) h->bits[i] = b[i];
        h->scale_mode = L.scale_mode;
        // s1_max_bits and wabs_max_bits were zeroed by the memset that precedes this kernel
    }
}

// One thread block per packed block (64 rows x one group).  Phase A: a warp per row computes the
// group's (s1, lo) and the top-width code of every element, in exactly the fp32 operation order of
// the definition (one IEEE rounding per operation, no contraction).  Phase B: the block assembles
// the segment words and writes them with coalesced stores.
// Calibrated packing (g_first >= 0 selects one group per launch): col_energy (optional) weights the scale fit of
// Eq. 5; err_out (optional, = W itself) receives, in place of the group's weights, their error at the top width
// divided by hc_diag[column] - the E of Algorithm 1 that the caller then takes out of the later columns.
__global__ void __launch_bounds__(PACK_THREADS)
pack_kernel(PackLayout L, const float* __restrict__ W, uint8_t* __restrict__ packed, int g_first,
            const float* __restrict__ col_energy, float* err_out, const float* __restrict__ hc_diag) {
    extern __shared__ uint8_t smem[];
    uint8_t* codes = smem;                                  // [64][g]
    const int G = (g_first >= 0 ? g_first : 0) + blockIdx.x, rt = blockIdx.y;
    const int g = L.g;
    uint8_t* blk = packed + d2moe_block_offset(L, rt, G);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float levels = (float)((1 << L.b1) - 1);
    unsigned s1_max_local = 0, wabs_max_local = 0;

    for (int r = warp; r < D2MOE_TILE_ROWS; r += PACK_THREADS / 32) {
        const long long row = (long long)rt * D2MOE_TILE_ROWS + r;
        if (row >= L.rows) {                                // padding rows: zero codes, zero meta
            for (int k = lane; k < g; k += 32) codes[r * g + k] = 0;
            if (lane == 0) {
                reinterpret_cast<uint32_t*>(blk)[r] = 0u;
                if (L.scale_mode == 1)
                    for (int l = 0; l < L.top - L.b1; ++l) *reinterpret_cast<uint16_t*>(blk + d2moe_level_offset(L, l, r)) = 0;
            }
            continue;
        }
        const float* src = W + row * (long long)L.cols + (long long)G * g;
        float wmin = INFINITY, wmax = -INFINITY;
        for (int k = lane; k < g; k += 32) { float v = src[k]; wmin = fminf(wmin, v); wmax = fmaxf(wmax, v); }
        for (int off = 16; off; off >>= 1) {
            wmin = fminf(wmin, __shfl_xor_sync(0xffffffffu, wmin, off));
            wmax = fmaxf(wmax, __shfl_xor_sync(0xffffffffu, wmax, off));
        }
        const __half lo_h = __float2half_rd(wmin);
        const float lo = __half2float(lo_h);
        __half s1_h = __float2half_ru(__fdiv_rn(__fsub_rn(wmax, lo), levels));
        float s1 = __half2float(s1_h);
        if (s1 == 0.0f) { s1 = 6.103515625e-05f; s1_h = __float2half_rn(s1); }   // 2^-14
        if (L.scale_mode == 0) {
            for (int k = lane; k < g; k += 32) {
                const float w = src[k];
                float q = rintf(__fdiv_rn(__fsub_rn(w, lo), s1));
                q = fminf(fmaxf(q, 0.0f), levels);
                float what = __fadd_rn(lo, __fmul_rn(q, s1));
                float res = __fsub_rn(w, what);
                int code = (int)q;
                float sj = __fmul_rn(s1, 0.25f);                 // s_1 = s1 * 2^-2
                for (int j = 1; j <= L.top - L.b1; ++j) {
                    const bool bit = res >= 0.0f;
                    what = __fadd_rn(what, bit ? sj : -sj);
                    res = __fsub_rn(w, what);
                    code = code * 2 + (bit ? 1 : 0);
                    sj = __fmul_rn(sj, 0.5f);
                }
                codes[r * g + k] = (uint8_t)code;
            }
        } else {
            // free per-step scales: every step needs the group's mean absolute residual first, so the lane keeps
            // its elements (k = lane, lane + 32, ...: at most 8) in registers and the steps run over the whole group
            float wv[8], wh[8], rs[8];
            int cd[8];
            const int n_el = g >> 5;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                if (e < n_el) {
                    const float w = src[lane + 32 * e];
                    float q = rintf(__fdiv_rn(__fsub_rn(w, lo), s1));
                    q = fminf(fmaxf(q, 0.0f), levels);
                    wv[e] = w;
                    wh[e] = __fadd_rn(lo, __fmul_rn(q, s1));
                    rs[e] = __fsub_rn(w, wh[e]);
                    cd[e] = (int)q;
                }
            }
            // Eq. 5 with per-column activation energies: the weighted mean of |R| (denominator: the group's energy sum)
            float dw[8], den = (float)g;
            if (col_energy) {
                float dpart = 0.0f;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    dw[e] = e < n_el ? col_energy[(long long)G * g + lane + 32 * e] : 0.0f;
                    if (e < n_el) dpart = __fadd_rn(dpart, dw[e]);
                }
                for (int off = 16; off; off >>= 1) dpart = __fadd_rn(dpart, __shfl_xor_sync(0xffffffffu, dpart, off));
                den = dpart;
            }
            for (int j = 1; j <= L.top - L.b1; ++j) {
                // mean |R| in the pinned order: this lane's elements ascending, then the butterfly
                float part = 0.0f;
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if (e < n_el) part = __fadd_rn(part, col_energy ? __fmul_rn(fabsf(rs[e]), dw[e]) : fabsf(rs[e]));
                for (int off = 16; off; off >>= 1) part = __fadd_rn(part, __shfl_xor_sync(0xffffffffu, part, off));
                const __half sj_h = __float2half_rn(__fdiv_rn(part, den));
                const float sj = __half2float(sj_h);
                if (lane == 0) *reinterpret_cast<__half*>(blk + d2moe_level_offset(L, j - 1, r)) = sj_h;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    if (e < n_el) {
                        const bool bit = rs[e] >= 0.0f;
                        wh[e] = __fadd_rn(wh[e], bit ? sj : -sj);
                        rs[e] = __fsub_rn(wv[e], wh[e]);
                        cd[e] = cd[e] * 2 + (bit ? 1 : 0);
                    }
                }
            }
#pragma unroll
            for (int e = 0; e < 8; ++e)
                if (e < n_el) codes[r * g + lane + 32 * e] = (uint8_t)cd[e];
            if (err_out) {                                  // E = (W - W_hat) / H^c[j, j], in place of the group's weights
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    if (e < n_el) {
                        const long long col = (long long)G * g + lane + 32 * e;
                        err_out[row * (long long)L.cols + col] = __fdiv_rn(__fsub_rn(wv[e], wh[e]), hc_diag[col * (L.cols + 1)]);
                    }
                }
            }
        }
        if (lane == 0) {
            __half2 m = __halves2half2(s1_h, lo_h);          // low half = s1, high half = lo
            reinterpret_cast<__half2*>(blk)[r] = m;
            s1_max_local = max(s1_max_local, __float_as_uint(s1));
            wabs_max_local = max(wabs_max_local, __float_as_uint(fmaxf(fabsf(wmin), fabsf(wmax))));
        }
    }
    if (lane == 0 && s1_max_local) {
        atomicMax(&reinterpret_cast<PackHeader*>(packed)->s1_max_bits, s1_max_local);
        atomicMax(&reinterpret_cast<PackHeader*>(packed)->wabs_max_bits, wabs_max_local);
    }
    __syncthreads();

    for (int j = 0; j < L.n_seg; ++j) {
        const int sw = L.seg_sw[j], per = 32 / sw, cs = L.seg_cs[j];
        const int row_bytes = g * sw / 8;
        const int n_words = D2MOE_TILE_ROWS * row_bytes / 4;
        const unsigned mask = (1u << L.seg_w[j]) - 1u;
        uint32_t* dst = reinterpret_cast<uint32_t*>(blk + L.seg_off[j]);
        for (int wi = threadIdx.x; wi < n_words; wi += PACK_THREADS) {
            const int ob = wi * 4;
            const int c = ob / (D2MOE_TILE_ROWS * cs);
            const int rem = ob - c * D2MOE_TILE_ROWS * cs;
            const int r = rem / cs, within = rem - r * cs;
            const int m = (c * cs + within) >> 2;
            uint32_t word = 0;
            for (int ko = 0; ko < per; ++ko) {         // element m*per + 4u + i: byte {0,2,1,3}[i], bit sw*u
                const int u = ko >> 2, i = ko & 3;
                const int byte = ((i & 1) << 1) | (i >> 1);
                const uint32_t v = (codes[r * g + m * per + ko] >> L.seg_shift[j]) & mask;
                word |= v << (8 * byte + sw * u);
            }
            dst[wi] = word;
        }
    }
}

__global__ void unpack_kernel(PackLayout L, const uint8_t* __restrict__ packed, int bits,
                              uint8_t* __restrict__ codes, float* __restrict__ scale,
                              float* __restrict__ offset) {
    const long long n = (long long)L.rows * L.cols;
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < n;
         idx += (long long)gridDim.x * blockDim.x) {
        const int row = (int)(idx / L.cols), col = (int)(idx - (long long)row * L.cols);
        const int rt = row / D2MOE_TILE_ROWS, r = row - rt * D2MOE_TILE_ROWS;
        const int G = col / L.g, k = col - G * L.g;
        const uint8_t* blk = packed + d2moe_block_offset(L, rt, G);
        unsigned code = 0;
        for (int j = 0; j < L.n_seg; ++j) {
            int bitpos;
            const int wo = d2moe_elem_word(L, j, r, k, &bitpos);
            const uint32_t word = *reinterpret_cast<const uint32_t*>(blk + wo);
            code |= ((word >> bitpos) & ((1u << L.seg_w[j]) - 1u)) << L.seg_shift[j];
        }
        codes[idx] = (uint8_t)(code >> (L.top - bits));
        if (k == 0) {
            const __half2 m = reinterpret_cast<const __half2*>(blk)[r];
            if (scale) scale[(long long)row * L.n_groups + G] = __low2float(m);
            if (offset) offset[(long long)row * L.n_groups + G] = __high2float(m);
        }
    }
}

// scale_mode 1: the free scale of every residual step, s_extra[row, G, level]
__global__ void unpack_scales_kernel(PackLayout L, const uint8_t* __restrict__ packed, float* __restrict__ s_extra) {
    const int n_lv = L.top - L.b1;
    const long long n = (long long)L.rows * L.n_groups * n_lv;
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < n;
         idx += (long long)gridDim.x * blockDim.x) {
        const int l = (int)(idx % n_lv);
        const long long rg = idx / n_lv;
        const int G = (int)(rg % L.n_groups), row = (int)(rg / L.n_groups);
        const int rt = row / D2MOE_TILE_ROWS, r = row - rt * D2MOE_TILE_ROWS;
        const uint8_t* blk = packed + d2moe_block_offset(L, rt, G);
        s_extra[idx] = __half2float(*reinterpret_cast<const __half*>(blk + d2moe_level_offset(L, l, r)));
    }
}

// Algorithm 1's propagation of a block's error: W[r, c] -= sum_j E[r, j] H^c[b + j, c] for every later column c,
// as g successive corrections in ascending j, each one fp32 multiply and one fp32 subtract (the oracle's order).
// E sits in W's own columns [b, b + g).  One thread per (row, column); the block's E rows are staged in shared memory.
__global__ void __launch_bounds__(256)
compensate_kernel(float* W, long long rows, int cols, int b, int g, const float* __restrict__ hc) {
    extern __shared__ float s_e[];                          // [16 rows][g]
    const int c = b + g + blockIdx.x * 16 + (threadIdx.x & 15);
    const long long r0 = (long long)blockIdx.y * 16;
    for (int i = threadIdx.x; i < 16 * g; i += 256) {
        const long long r = r0 + i / g;
        s_e[i] = r < rows ? W[r * cols + b + (i % g)] : 0.0f;
    }
    __syncthreads();
    const long long r = r0 + (threadIdx.x >> 4);
    if (r >= rows || c >= cols) return;
    float acc = W[r * cols + c];
    const float* e = s_e + (threadIdx.x >> 4) * g;
    for (int j = 0; j < g; ++j) acc = __fsub_rn(acc, __fmul_rn(e[j], hc[(long long)(b + j) * cols + c]));
    W[r * cols + c] = acc;
}

}  // namespace

cudaError_t launch_pack_calibrated(const PackLayout& L, const int* bits, int n_bits, float* W, const float* hc,
                                   const float* col_energy, uint8_t* packed, cudaStream_t st) {
    cudaError_t err = cudaMemsetAsync(packed, 0, D2MOE_HEADER_BYTES, st);
    if (err != cudaSuccess) return err;
    int b[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int i = 0; i < n_bits; ++i) b[i] = bits[i];
    pack_header_kernel<<<1, 32, 0, st>>>(reinterpret_cast<PackHeader*>(packed), L, n_bits,
                                         b[0], b[1], b[2], b[3], b[4], b[5], b[6], b[7]);
    const size_t smem = (size_t)D2MOE_TILE_ROWS * L.g;
    for (int G = 0; G < L.n_groups; ++G) {
        const bool prop = hc != nullptr && G + 1 < L.n_groups;
        dim3 grid(1, L.n_rt);
        pack_kernel<<<grid, PACK_THREADS, smem, st>>>(L, W, packed, G, col_energy, prop ? W : nullptr, hc);
        if (prop) {
            const int later = L.cols - (G + 1) * L.g;
            dim3 cg((later + 15) / 16, (unsigned)((L.rows + 15) / 16));
            compensate_kernel<<<cg, 256, (size_t)16 * L.g * 4, st>>>(W, L.rows, L.cols, G * L.g, L.g, hc);
        }
    }
    return cudaGetLastError();
}

cudaError_t launch_unpack_scales(const PackLayout& L, const uint8_t* packed, float* s_extra, cudaStream_t st) {
    const long long n = (long long)L.rows * L.n_groups * (L.top - L.b1);
    if (n == 0) return cudaSuccess;
    int blocks = (int)((n + 255) / 256 < 148 * 16 ? (n + 255) / 256 : 148 * 16);
    unpack_scales_kernel<<<blocks, 256, 0, st>>>(L, packed, s_extra);
    return cudaGetLastError();
}

cudaError_t launch_pack(const PackLayout& L, const int* bits, int n_bits, const float* W, uint8_t* packed,
                        cudaStream_t st) {
    cudaError_t err = cudaMemsetAsync(packed, 0, D2MOE_HEADER_BYTES, st);
    if (err != cudaSuccess) return err;
    int b[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int i = 0; i < n_bits; ++i) b[i] = bits[i];
    pack_header_kernel<<<1, 32, 0, st>>>(reinterpret_cast<PackHeader*>(packed), L, n_bits,
                                         b[0], b[1], b[2], b[3], b[4], b[5], b[6], b[7]);
    dim3 grid(L.n_groups, L.n_rt);
    size_t smem = (size_t)D2MOE_TILE_ROWS * L.g;
    pack_kernel<<<grid, PACK_THREADS, smem, st>>>(L, W, packed, -1, nullptr, nullptr, nullptr);
    return cudaGetLastError();
}

cudaError_t launch_unpack(const PackLayout& L, const uint8_t* packed, int bits, uint8_t* codes,
                          float* scale, float* offset, cudaStream_t st) {
    long long n = (long long)L.rows * L.cols;
    int blocks = (int)((n + 255) / 256 < 148 * 16 ? (n + 255) / 256 : 148 * 16);
    if (blocks < 1) blocks = 1;
    unpack_kernel<<<blocks, 256, 0, st>>>(L, packed, bits, codes, scale, offset);
    return cudaGetLastError();
}
