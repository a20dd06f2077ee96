// Plain CUDA-core expert kernels: every (assignment, output row) is one warp's fp32 dot product over
// weights dequantized on the fly at the assignment's routed width (Section 3.3.1 reconstruction
// rule, in its closed form W_hat_b = (lo - s1/2) + s_b (q_b + 1/2), s_b = s1 / 2^(b-b1)).
// Works for every supported shape; it is the path of last resort and the on-device cross-check of
// the tensor-core kernels.  Also: the weighted combine (with optional residual) and RMSNorm.
#include "d2moe_common.cuh"
#include <cstdint>

namespace {

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

// Resolve assignment id a (routed: a < A; shared experts after) into token, expert, width index.
__device__ __forceinline__ bool resolve_assignment(const MoeDims& D, const RouteBufs& R, int a, int* t,
                                                   int* e, int* kk, int32_t* device_status) {
    if (a < D.A) {
        *t = a / D.k;
        *e = R.topk_idx[a];
        *kk = R.bit_idx[a];
        if (*e < 0 || *e >= D.E || *kk < 0 || *kk >= D.K) {
            if (device_status) atomicOr(device_status, D2MOE_DEV_BAD_INDEX);
            return false;
        }
    } else {
        const int s = (a - D.A) / D.T;
        *t = (a - D.A) - s * D.T;
        *e = D.E + s;
        *kk = D.K - 1;
    }
    return true;
}

// Dot product of packed row `row` of one matrix, read at width index kk, with vector v (length
// L.cols).  All 32 lanes take part; the result is valid in every lane.
template <typename VT>
__device__ float row_dot(const PackLayout& L, const uint8_t* __restrict__ packed, int row, int kk,
                         const VT* __restrict__ v, int lane) {
    const int rt = row / D2MOE_TILE_ROWS, r = row - rt * D2MOE_TILE_ROWS;
    const int last = L.last_seg[kk];                    // the call reads stored segments 0..last
    const int b = L.seg_shift[last];                    // top - bits[kk]
    const int width = L.top - b;
    const float inv = 1.0f / (float)(1 << (width - L.b1));
    float acc = 0.0f;
    for (int G = 0; G < L.n_groups; ++G) {
        const uint8_t* blk = packed + d2moe_block_offset(L, rt, G);
        const __half2 m = reinterpret_cast<const __half2*>(blk)[r];
        const float s1 = __low2float(m), lo = __high2float(m);
        const float sb = s1 * inv;
        const float base = lo - 0.5f * s1;
        const VT* vg = v + (size_t)G * L.g;
        // free residual scales (Eq. 4 / Eq. 5): the additive rule W_hat = lo + s1 Q + sum over the steps of (+-) s_l
        const int n_lv = width - L.b1;
        float sl[7];
        if (L.scale_mode == 1) {
#pragma unroll
            for (int l = 0; l < 7; ++l)
                sl[l] = l < n_lv ? __half2float(*reinterpret_cast<const __half*>(blk + d2moe_level_offset(L, l, r))) : 0.0f;
        }
        for (int i = lane; i < L.g / 2; i += 32) {      // pair (2i, 2i+1)
            unsigned q0 = 0, q1 = 0;
            for (int j = 0; j <= last; ++j) {
                int bitpos;
                const int wo = d2moe_elem_word(L, j, r, 2 * i, &bitpos);
                const uint32_t word = *reinterpret_cast<const uint32_t*>(blk + wo);
                const unsigned mask = (1u << L.seg_w[j]) - 1u;
                q0 |= ((word >> bitpos) & mask) << L.seg_shift[j];
                q1 |= ((word >> (bitpos + 16)) & mask) << L.seg_shift[j];
            }
            q0 >>= b; q1 >>= b;
            float w0, w1;
            if (L.scale_mode == 1) {
                w0 = fmaf(s1, (float)(q0 >> n_lv), lo);
                w1 = fmaf(s1, (float)(q1 >> n_lv), lo);
#pragma unroll
                for (int l = 0; l < 7; ++l) {
                    if (l < n_lv) {
                        w0 += ((q0 >> (n_lv - 1 - l)) & 1u) ? sl[l] : -sl[l];
                        w1 += ((q1 >> (n_lv - 1 - l)) & 1u) ? sl[l] : -sl[l];
                    }
                }
            } else {
                w0 = fmaf(sb, (float)q0 + 0.5f, base);
                w1 = fmaf(sb, (float)q1 + 0.5f, base);
            }
            acc = fmaf(w0, to_f32(vg[2 * i]), acc);
            acc = fmaf(w1, to_f32(vg[2 * i + 1]), acc);
        }
    }
    for (int off = 16; off; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    return acc;
}

// h[a, r] = silu(Wg_{e,b}[r,:] . x_t) * (Wu_{e,b}[r,:] . x_t);  grid (A_tot, ceil(F/8)), 8 warps.
__global__ void __launch_bounds__(256)
gateup_cc_kernel(MoeDims D, PackLayout L, ExpertPtrs P, const __nv_bfloat16* __restrict__ x, RouteBufs R,
                 float* __restrict__ hbuf, int32_t* device_status) {
    pdl_enter();
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.y * 8 + (threadIdx.x >> 5);
    const int a = blockIdx.x;                       // assignments on the x dimension: no 65535 limit
    if (row >= D.F) return;
    int t, e, kk;
    if (!resolve_assignment(D, R, a, &t, &e, &kk, device_status)) {
        if (lane == 0) hbuf[(size_t)a * D.F + row] = 0.0f;
        return;
    }
    const __nv_bfloat16* xt = x + (size_t)t * D.d;
    const float g = row_dot(L, P.w[3 * e + 0], row, kk, xt, lane);
    const float u = row_dot(L, P.w[3 * e + 1], row, kk, xt, lane);
    if (lane == 0) hbuf[(size_t)a * D.F + row] = g / (1.0f + expf(-g)) * u;
}

// o[a, r] = Wd_{e,b}[r,:] . h[a,:];  grid (A_tot, ceil(d/8))
__global__ void __launch_bounds__(256)
down_cc_kernel(MoeDims D, PackLayout L, ExpertPtrs P, RouteBufs R, const float* __restrict__ hbuf,
               float* __restrict__ obuf, int32_t* device_status) {
    pdl_enter();
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.y * 8 + (threadIdx.x >> 5);
    const int a = blockIdx.x;
    if (row >= D.d) return;
    int t, e, kk;
    if (!resolve_assignment(D, R, a, &t, &e, &kk, nullptr)) {
        if (lane == 0) obuf[(size_t)a * D.d + row] = 0.0f;
        return;
    }
    const float o = row_dot(L, P.w[3 * e + 2], row, kk, hbuf + (size_t)a * D.F, lane);
    if (lane == 0) obuf[(size_t)a * D.d + row] = o;
}

// y[t, c] = bf16( residual[t, c] + sum_slot w[t,slot] * o[row(t,slot), c] + sum_shared o[...] )
// where o may come as n_split partial sums (split-K); row_map (optional) maps an assignment id to
// its row in obuf.
__global__ void combine_kernel(MoeDims D, RouteBufs R, const float* __restrict__ obuf, int n_split,
                               size_t split_stride, const int32_t* __restrict__ row_map,
                               const __nv_bfloat16* __restrict__ residual, __nv_bfloat16* __restrict__ y) {
    pdl_enter();
    const int t = blockIdx.x;                       // tokens on the x dimension: no 65535 limit
    const int c = blockIdx.y * blockDim.x + threadIdx.x;
    if (c >= D.d) return;
    float acc = residual ? __bfloat162float(residual[(size_t)t * D.d + c]) : 0.0f;
    float sum = 0.0f;
    for (int s = 0; s < D.k + D.n_shared; ++s) {
        const int a = s < D.k ? t * D.k + s : D.A + (s - D.k) * D.T + t;
        const float w = s < D.k ? R.topk_w[a] : 1.0f;
        const long long rowi = row_map ? (long long)row_map[a] : (long long)a;
        if (rowi < 0) continue;                      // an assignment that was skipped (bad routing index)
        const size_t row = (size_t)rowi;
        float o = 0.0f;
        for (int sp = 0; sp < n_split; ++sp) o += obuf[sp * split_stride + row * D.d + c];
        sum = fmaf(w, o, sum);
    }
    y[(size_t)t * D.d + c] = __float2bfloat16_rn(acc + sum);
}

// The same, four columns per thread (16-byte loads of the partial outputs, 8-byte loads / stores of the
// bf16 rows); every element is summed in the same order as above.  Needs d % 4 == 0.
__global__ void combine4_kernel(MoeDims D, RouteBufs R, const float* __restrict__ obuf, int n_split,
                                size_t split_stride, const int32_t* __restrict__ row_map,
                                const __nv_bfloat16* __restrict__ residual, __nv_bfloat16* __restrict__ y) {
    pdl_enter();
    const int t = blockIdx.x;
    const int c = 4 * (blockIdx.y * blockDim.x + threadIdx.x);
    if (c >= D.d) return;
    float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    if (residual) {
        const uint2 rv = *reinterpret_cast<const uint2*>(residual + (size_t)t * D.d + c);
        const __nv_bfloat162 r01 = *reinterpret_cast<const __nv_bfloat162*>(&rv.x);
        const __nv_bfloat162 r23 = *reinterpret_cast<const __nv_bfloat162*>(&rv.y);
        acc[0] = __low2float(r01); acc[1] = __high2float(r01); acc[2] = __low2float(r23); acc[3] = __high2float(r23);
    }
    float sum[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    for (int s = 0; s < D.k + D.n_shared; ++s) {
        const int a = s < D.k ? t * D.k + s : D.A + (s - D.k) * D.T + t;
        const float w = s < D.k ? R.topk_w[a] : 1.0f;
        const long long rowi = row_map ? (long long)row_map[a] : (long long)a;
        if (rowi < 0) continue;                      // an assignment that was skipped (bad routing index)
        const size_t row = (size_t)rowi;
        float o[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        for (int sp = 0; sp < n_split; ++sp) {
            const float4 v = *reinterpret_cast<const float4*>(obuf + sp * split_stride + row * D.d + c);
            o[0] += v.x; o[1] += v.y; o[2] += v.z; o[3] += v.w;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) sum[i] = fmaf(w, o[i], sum[i]);
    }
    __nv_bfloat162 y01, y23;
    y01.x = __float2bfloat16_rn(acc[0] + sum[0]); y01.y = __float2bfloat16_rn(acc[1] + sum[1]);
    y23.x = __float2bfloat16_rn(acc[2] + sum[2]); y23.y = __float2bfloat16_rn(acc[3] + sum[3]);
    uint2 out;
    out.x = *reinterpret_cast<const uint32_t*>(&y01);
    out.y = *reinterpret_cast<const uint32_t*>(&y23);
    *reinterpret_cast<uint2*>(y + (size_t)t * D.d + c) = out;
}

// xn = bf16( x / sqrt(mean(x^2) + eps) ), fp64 inside so the rounding matches a double-precision
// evaluation; one block per token.
__global__ void __launch_bounds__(256)
rmsnorm_kernel(int d, double eps, const __nv_bfloat16* __restrict__ x, __nv_bfloat16* __restrict__ xn) {
    pdl_enter();
    __shared__ double red[8];
    const int t = blockIdx.x;
    double ss = 0.0;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        const double v = (double)__bfloat162float(x[(size_t)t * d + i]);
        ss += v * v;
    }
    for (int off = 16; off; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    double tot = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += red[w];
    const double inv = 1.0 / sqrt(tot / (double)d + eps);
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        const double v = (double)__bfloat162float(x[(size_t)t * d + i]) * inv;
        xn[(size_t)t * d + i] = __float2bfloat16_rn((float)v);
    }
}

}  // namespace

cudaError_t launch_gateup_cuda_core(const MoeDims& D, const PackLayout& Lgu, const ExpertPtrs& P,
                                    const __nv_bfloat16* x, const RouteBufs& R, float* hbuf,
                                    int32_t* device_status, cudaStream_t st) {
    if (D.A_tot == 0) return cudaSuccess;
    dim3 g1(D.A_tot, (D.F + 7) / 8);
    launch_chained(gateup_cc_kernel, dim3(g1), dim3(256), 0, st, D, Lgu, P, x, R, hbuf, device_status);
    return cudaGetLastError();
}

cudaError_t launch_down_cuda_core(const MoeDims& D, const PackLayout& Ld, const ExpertPtrs& P,
                                  const RouteBufs& R, const float* hbuf, float* obuf,
                                  int32_t* device_status, cudaStream_t st) {
    if (D.A_tot == 0) return cudaSuccess;
    dim3 g2(D.A_tot, (D.d + 7) / 8);
    launch_chained(down_cc_kernel, dim3(g2), dim3(256), 0, st, D, Ld, P, R, hbuf, obuf, device_status);
    return cudaGetLastError();
}

cudaError_t launch_combine(const MoeDims& D, const RouteBufs& R, const float* obuf, int n_split,
                           size_t split_stride, const int32_t* row_map, const __nv_bfloat16* residual,
                           __nv_bfloat16* y, cudaStream_t st) {
    if (D.T == 0) return cudaSuccess;
    const bool vec = D.d % 4 == 0 && split_stride % 4 == 0 && ((uintptr_t)obuf & 15) == 0 && ((uintptr_t)y & 7) == 0 &&
                     ((uintptr_t)residual & 7) == 0;
    if (vec) {
        dim3 grid(D.T, (D.d / 4 + 127) / 128);
        launch_chained(combine4_kernel, dim3(grid), dim3(128), 0, st, D, R, obuf, n_split, split_stride, row_map, residual, y);
    } else {
        dim3 grid(D.T, (D.d + 255) / 256);
        launch_chained(combine_kernel, dim3(grid), dim3(256), 0, st, D, R, obuf, n_split, split_stride, row_map, residual, y);
    }
    return cudaGetLastError();
}

cudaError_t launch_rmsnorm(int T, int d, float eps, const __nv_bfloat16* x, __nv_bfloat16* xn, cudaStream_t st) {
    if (T == 0) return cudaSuccess;
    launch_chained(rmsnorm_kernel, dim3(T), dim3(256), 0, st, d, (double)eps, x, xn);
    return cudaGetLastError();
}
