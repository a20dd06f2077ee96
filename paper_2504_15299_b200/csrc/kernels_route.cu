// Dual routing (expert gate top-k + per-expert bit-width choice, Section 3.2) and the stable
// grouping of assignments by (expert, width); its histogram is B_{j,k} of Section 3.4.3.
#include "d2moe_common.cuh"
#include "tc_common.cuh"
#include "group_block.cuh"

namespace {

constexpr int MAX_TOPK = 8;
constexpr int MAX_E_PER_LANE = 8;        // up to 256 experts

// fp32 dot product in the pinned order: lane l accumulates elements l, l+32, ... with one fused
// multiply-add each, then a butterfly reduction with offsets 16, 8, 4, 2, 1.
__device__ __forceinline__ float dot_pinned(const __nv_bfloat16* __restrict__ a,
                                            const __nv_bfloat16* __restrict__ b, int d, int lane) {
    float acc = 0.0f;
    for (int i = lane; i < d; i += 32)
        acc = fmaf(__bfloat162float(a[i]), __bfloat162float(b[i]), acc);
    for (int off = 16; off; off >>= 1) acc = acc + __shfl_xor_sync(0xffffffffu, acc, off);
    return acc;
}

// One warp: the gate of one token from its logits (lane l holds the logits of experts l, l + 32, ...).
// k rounds of arg-max over the remaining logits, ties to the lower index (shuffle reduction); softmax over
// all experts, gathered at the selected ones.  Outputs in every lane: sel[s], w[s] (not renormalised) and
// their sum; a NaN or an infinity among the logits raises D2MOE_DEV_NONFINITE.
__device__ __forceinline__ void gate_select(const float (&lg)[MAX_E_PER_LANE], int E, int k, int lane,
                                            int (&sel)[MAX_TOPK], float (&w)[MAX_TOPK], float& wsum,
                                            int32_t* __restrict__ device_status) {
    bool bad = false;
#pragma unroll
    for (int m = 0; m < MAX_E_PER_LANE; ++m)
        if (lane + 32 * m < E && !isfinite(lg[m])) bad = true;
    if (__any_sync(0xffffffffu, bad) && lane == 0 && device_status) atomicOr(device_status, D2MOE_DEV_NONFINITE);

    unsigned taken = 0;
    float selv[MAX_TOPK];
#pragma unroll
    for (int s = 0; s < MAX_TOPK; ++s) {
        sel[s] = 0; selv[s] = 0.0f;
        if (s < k) {
            float bv = -INFINITY; int bi = 0x7fffffff;
#pragma unroll
            for (int m = 0; m < MAX_E_PER_LANE; ++m) {
                const int e = lane + 32 * m;
                if (e < E && !((taken >> m) & 1u)) {
                    if (bi == 0x7fffffff || lg[m] > bv) { bv = lg[m]; bi = e; }
                }
            }
            for (int off = 16; off; off >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
                const bool take = (oi != 0x7fffffff) &&
                                  (bi == 0x7fffffff || ov > bv || (ov == bv && oi < bi));
                if (take) { bv = ov; bi = oi; }
            }
            sel[s] = bi; selv[s] = bv;
            if ((bi & 31) == lane) taken |= 1u << (bi >> 5);
        }
    }
    const float mx = selv[0];
    float part = 0.0f;
#pragma unroll
    for (int m = 0; m < MAX_E_PER_LANE; ++m)
        if (lane + 32 * m < E) part += expf(lg[m] - mx);
    for (int off = 16; off; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
    wsum = 0.0f;
#pragma unroll
    for (int s = 0; s < MAX_TOPK; ++s) {
        w[s] = 0.0f;
        if (s < k) { w[s] = expf(selv[s] - mx) / part; wsum += w[s]; }
    }
}

// One warp per token.
__global__ void __launch_bounds__(128)
route_kernel(MoeDims D, const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ gate_w,
             const float* __restrict__ logits_in, const __nv_bfloat16* __restrict__ bit_w,
             const int8_t* __restrict__ forced, RouteBufs R, int32_t* __restrict__ keys,
             int32_t* __restrict__ device_status) {
    pdl_enter();
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= D.T) return;
    const int E = D.E;
    const __nv_bfloat16* xt = x + (size_t)t * D.d;

    float lg[MAX_E_PER_LANE];
#pragma unroll
    for (int m = 0; m < MAX_E_PER_LANE; ++m) lg[m] = -INFINITY;
    if (logits_in) {
#pragma unroll
        for (int m = 0; m < MAX_E_PER_LANE; ++m) {
            const int e = lane + 32 * m;
            if (e < E) lg[m] = logits_in[(size_t)t * E + e];
        }
    } else {
        for (int e = 0; e < E; ++e) {
            const float v = dot_pinned(xt, gate_w + (size_t)e * D.d, D.d, lane);
#pragma unroll
            for (int m = 0; m < MAX_E_PER_LANE; ++m)
                if (m == (e >> 5) && lane == (e & 31)) lg[m] = v;
        }
    }
    int sel[MAX_TOPK];
    float w[MAX_TOPK];
    float wsum;
    gate_select(lg, E, D.k, lane, sel, w, wsum, device_status);

    // bit-width choice per selected expert
#pragma unroll
    for (int s = 0; s < MAX_TOPK; ++s) {
        if (s < D.k) {
            const int a = t * D.k + s;
            int kk;
            if (forced) {
                kk = forced[a];
                if (kk < 0 || kk >= D.K) {
                    if (lane == 0 && device_status) atomicOr(device_status, D2MOE_DEV_BAD_INDEX);
                    kk = kk < 0 ? 0 : D.K - 1;
                }
            } else {
                float best = 0.0f; kk = 0;
                for (int c = 0; c < D.K; ++c) {
                    const float u = dot_pinned(xt, bit_w + ((size_t)sel[s] * D.K + c) * D.d, D.d, lane);
                    if (c == 0 || u > best) { best = u; kk = c; }
                }
            }
            if (lane == 0) {
                R.topk_idx[a] = sel[s];
                R.topk_w[a] = D.renormalize ? w[s] / wsum : w[s];
                R.bit_idx[a] = (int8_t)kk;
                keys[a] = sel[s] * D.K + kk;
            }
        }
    }
}

// One warp per key: count the assignments that carry it.
__global__ void count_kernel(int A, int n_keys, const int32_t* __restrict__ keys, int32_t* __restrict__ hist) {
    pdl_enter();
    const int lane = threadIdx.x & 31;
    const int key = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (key >= n_keys) return;
    int cnt = 0;
    for (int base = 0; base < A; base += 32) {
        const int a = base + lane;
        const bool m = a < A && keys[a] == key;
        cnt += __popc(__ballot_sync(0xffffffffu, m));
    }
    if (lane == 0) hist[key] = cnt;
}

// Exclusive prefix sum of the histogram by one warp.
__global__ void scan_kernel(int n_keys, const int32_t* __restrict__ hist, int32_t* __restrict__ group_off) {
    pdl_enter();
    const int lane = threadIdx.x;
    int carry = 0;
    for (int base = 0; base < n_keys; base += 32) {
        const int i = base + lane;
        const int v = i < n_keys ? hist[i] : 0;
        int incl = v;
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += o;
        }
        if (i < n_keys) group_off[i] = carry + incl - v;
        carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) group_off[n_keys] = carry;
}

// One warp per key: write its assignments, in ascending assignment id, from group_off[key] on.
__global__ void scatter_kernel(int A, int n_keys, const int32_t* __restrict__ keys,
                               const int32_t* __restrict__ group_off, int32_t* __restrict__ perm,
                               int32_t* __restrict__ inv_perm) {
    pdl_enter();
    const int lane = threadIdx.x & 31;
    const int key = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (key >= n_keys) return;
    int pos = group_off[key];
    const int end = group_off[key + 1];
    if (pos == end) return;
    for (int base = 0; base < A; base += 32) {
        const int a = base + lane;
        const bool m = a < A && keys[a] == key;
        const unsigned bal = __ballot_sync(0xffffffffu, m);
        if (m) {
            const int p = pos + __popc(bal & ((1u << lane) - 1u));
            perm[p] = a;
            inv_perm[a] = p;
        }
        pos += __popc(bal);
    }
}

// Small and mid-sized loads: histogram, scan and scatter in one launch.  Every block stages all keys in shared
// memory and counts every key itself (32 warps, a key per warp at a time), so no block waits for another;
// block b then writes the groups of the keys b, b + grid, ...  One block for decode-sized loads, a few
// blocks for a prefill batch of a few thousand assignments on a few dozen keys.  Same warp-per-key ballot
// walks as the three kernels above: the same stable order.  smem: A keys + n_keys + 1 ints.
__global__ void __launch_bounds__(1024)
group_block_kernel(int A, int n_keys, const int32_t* __restrict__ keys, int32_t* __restrict__ group_off,
                 int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm) {
    pdl_enter();
    extern __shared__ int32_t s_grp[];
    group_block_body(A, n_keys, keys, group_off, perm, inv_perm, s_grp, blockIdx.x, gridDim.x);
}

// One block, counting sort: up to a few thousand assignments on up to 512 keys (see group_block.cuh).
__global__ void __launch_bounds__(1024)
group_sort_kernel(int A, int n_keys, const int32_t* __restrict__ keys, int32_t* __restrict__ group_off,
                  int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm) {
    pdl_enter();
    extern __shared__ int32_t s_grp[];
    group_sort_body(A, n_keys, keys, group_off, perm, inv_perm, s_grp);
}

// Same dot product with both vectors already in shared memory.
__device__ __forceinline__ float dot_pinned_smem(const __nv_bfloat16* a, const __nv_bfloat16* b, int d, int lane) {
    float acc = 0.0f;
#pragma unroll 8
    for (int i = lane; i < d; i += 32)
        acc = fmaf(__bfloat162float(a[i]), __bfloat162float(b[i]), acc);
    for (int off = 16; off; off >>= 1) acc = acc + __shfl_xor_sync(0xffffffffu, acc, off);
    return acc;
}

// Copies d elements (a multiple of 8; both ends 16-byte aligned) into shared memory with asynchronous 16-byte copies:
// every copy of a block is in flight at once (one trip to memory instead of one per few registers).  The data may
// be read after stage_wait() and a barrier.
__device__ __forceinline__ void stage_row(__nv_bfloat16* dst, const __nv_bfloat16* __restrict__ src, int d) {
    const uint4* s = reinterpret_cast<const uint4*>(src);
    const uint32_t t = smem_u32(dst);
    for (int i = threadIdx.x; i < d / 8; i += blockDim.x)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(t + 16u * (uint32_t)i), "l"(s + i) : "memory");
}
__device__ __forceinline__ void stage_wait() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Gate logits for many experts: a block stages TB token rows and EB weight rows once and forms the
// TB x EB dot products (pinned order), so a weight row is read once per TB tokens instead of per token.
__global__ void __launch_bounds__(256)
gate_logits_kernel(int T, int E, int d, const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ gate_w,
                   float* __restrict__ logits, int TB, int EB) {
    pdl_enter();
    extern __shared__ __align__(16) uint8_t rsm[];
    __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(rsm);
    __nv_bfloat16* ws = xs + (size_t)TB * d;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t0 = blockIdx.x * TB, e0 = blockIdx.y * EB;
    const int nt = min(TB, T - t0), ne = min(EB, E - e0);
    stage_row(xs, x + (size_t)t0 * d, nt * d);                 // consecutive rows are contiguous: one copy loop each
    stage_row(ws, gate_w + (size_t)e0 * d, ne * d);
    stage_wait();
    __syncthreads();
    for (int pr = warp; pr < nt * ne; pr += 8) {
        const int tt = pr / ne, ee = pr - tt * ne;
        const float v = dot_pinned_smem(xs + (size_t)tt * d, ws + (size_t)ee * d, d, lane);
        if (lane == 0) logits[(size_t)(t0 + tt) * E + e0 + ee] = v;
    }
}

// One block (8 warps) per token: the same results as route_kernel, with the token row and batches of
// EB weight rows staged in shared memory by 16-byte loads (the pinned summation order makes a lane
// walk a row with stride 32, which is slow straight from global memory); warp w takes row w of a batch.
__global__ void __launch_bounds__(256)
route_block_kernel(MoeDims D, const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ gate_w,
                   const float* __restrict__ logits_in, const __nv_bfloat16* __restrict__ bit_w,
                   const int8_t* __restrict__ forced, RouteBufs R, int32_t* __restrict__ keys,
                   int32_t* __restrict__ device_status, int EB) {
    pdl_enter();
    extern __shared__ __align__(16) uint8_t rsm[];
    __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(rsm);
    __nv_bfloat16* ws = xs + D.d;
    float* lg_s = reinterpret_cast<float*>(ws + (size_t)EB * D.d);     // [E]
    float* u_s = lg_s + D.E;                                             // [k * K]
    int* sel_s = reinterpret_cast<int*>(u_s + MAX_TOPK * 8);             // [k]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = blockIdx.x;
    const int E = D.E;

    if (!(logits_in && forced)) stage_row(xs, x + (size_t)t * D.d, D.d);
    if (logits_in) {
        for (int e = threadIdx.x; e < E; e += blockDim.x) lg_s[e] = logits_in[(size_t)t * E + e];
        stage_wait();
        __syncthreads();
    } else {
        for (int eb = 0; eb < E; eb += EB) {
            const int n = min(EB, E - eb);
            stage_row(ws, gate_w + (size_t)eb * D.d, n * D.d);       // the n rows are contiguous: one copy loop
            stage_wait();
            __syncthreads();
            for (int r = warp; r < n; r += 8) {
                const float v = dot_pinned_smem(xs, ws + (size_t)r * D.d, D.d, lane);
                if (lane == 0) lg_s[eb + r] = v;
            }
            __syncthreads();
        }
    }

    float w[MAX_TOPK];
    float wsum = 0.0f;
    int sel[MAX_TOPK];
    if (warp == 0) {
        float lg[MAX_E_PER_LANE];
#pragma unroll
        for (int m = 0; m < MAX_E_PER_LANE; ++m) {
            const int e = lane + 32 * m;
            lg[m] = e < E ? lg_s[e] : -INFINITY;
        }
        gate_select(lg, E, D.k, lane, sel, w, wsum, device_status);
        if (lane == 0) {
#pragma unroll
            for (int s = 0; s < MAX_TOPK; ++s)
                if (s < D.k) sel_s[s] = sel[s];
        }
    }
    __syncthreads();

    if (!forced) {              // bit-width router logits of the selected experts: rows (slot s, width c)
        const int n_rows = D.k * D.K;
        for (int rb = 0; rb < n_rows; rb += EB) {
            const int n = min(EB, n_rows - rb);
            for (int r = 0; r < n; ++r) {
                const int s = (rb + r) / D.K, c = (rb + r) - s * D.K;
                stage_row(ws + (size_t)r * D.d, bit_w + ((size_t)sel_s[s] * D.K + c) * D.d, D.d);
            }
            stage_wait();
            __syncthreads();
            for (int r = warp; r < n; r += 8) {
                const float v = dot_pinned_smem(xs, ws + (size_t)r * D.d, D.d, lane);
                if (lane == 0) u_s[rb + r] = v;
            }
            __syncthreads();
        }
    }

    if (warp == 0 && lane == 0) {
#pragma unroll
        for (int s = 0; s < MAX_TOPK; ++s) {
            if (s < D.k) {
                const int a = t * D.k + s;
                int kk = 0;
                if (forced) {
                    kk = forced[a];
                    if (kk < 0 || kk >= D.K) {
                        if (device_status) atomicOr(device_status, D2MOE_DEV_BAD_INDEX);
                        kk = kk < 0 ? 0 : D.K - 1;
                    }
                } else {
                    float best = u_s[s * D.K];
                    for (int c = 1; c < D.K; ++c)
                        if (u_s[s * D.K + c] > best) { best = u_s[s * D.K + c]; kk = c; }
                }
                R.topk_idx[a] = sel[s];
                R.topk_w[a] = D.renormalize ? w[s] / wsum : w[s];
                R.bit_idx[a] = (int8_t)kk;
                keys[a] = sel[s] * D.K + kk;
            }
        }
    }
}

}  // namespace

cudaError_t launch_route(const MoeDims& D, const __nv_bfloat16* x, const __nv_bfloat16* gate_w,
                         const float* logits_in, const __nv_bfloat16* bit_w, const int8_t* forced,
                         const RouteBufs& R, float* logits_ws, int32_t* keys_ws, int32_t* hist_ws,
                         int32_t* device_status, cudaStream_t st, bool* defer_small_group) {
    const int warps_per_block = 4;
    const int n_keys = D.E * D.K;
    // block-per-token kernel when the token row plus at least one weight row fit in shared memory
    const size_t row_bytes = (size_t)D.d * 2;
    const size_t tail_bytes = (size_t)(D.E + MAX_TOPK * 8 + MAX_TOPK) * 4 + 64;
    const size_t budget = 200 * 1024;
    int EB = row_bytes + tail_bytes < budget ? (int)((budget - row_bytes - tail_bytes) / row_bytes) : 0;
    if (EB > 8) EB = 8;
    if (EB >= 1 && D.d % 8 == 0) {
        // many experts: gate logits by the tiled kernel first, then route from those logits
        if (!logits_in && D.E > 16 && logits_ws && 16 * row_bytes <= budget) {
            const int TB = 8, EBL = 8;
            const size_t lsm = (size_t)(TB + EBL) * row_bytes;
            cudaError_t e = ensure_dynamic_smem<&gate_logits_kernel>((int)lsm);
            if (e != cudaSuccess) return e;
            dim3 grid((D.T + TB - 1) / TB, (D.E + EBL - 1) / EBL);
            launch_chained(gate_logits_kernel, dim3(grid), dim3(256), lsm, st, D.T, D.E, D.d, x, gate_w, logits_ws, TB, EBL);
            logits_in = logits_ws;
            gate_w = nullptr;
        }
        const size_t smem = row_bytes * (1 + EB) + tail_bytes;
        cudaError_t e = ensure_dynamic_smem<&route_block_kernel>((int)smem);
        if (e != cudaSuccess) return e;
        // logits and widths both supplied: no dot products, one warp per token does the selection
        const int threads = (logits_in && forced) ? 32 : 256;
        launch_chained(route_block_kernel, dim3(D.T), dim3(threads), smem, st, D, x, gate_w, logits_in, bit_w, forced, R, keys_ws, device_status, EB);
    } else
    launch_chained(route_kernel, dim3((D.T + warps_per_block - 1) / warps_per_block), dim3(warps_per_block * 32), 0, st, 
        D, x, gate_w, logits_in, bit_w, forced, R, keys_ws, device_status);
    // few assignments and keys: histogram, scan and scatter in one single-block launch (beyond about a
    // thousand warp walks the three grid-wide kernels are faster: 39 vs 10 us at 192 keys x 1536 assignments)
    const bool small = d2moe_group_is_small(D.A, n_keys);
    // the caller runs the single-block grouping in front of its next kernel (one launch instead of two)
    if ((small || d2moe_group_is_sortable(D.A, n_keys)) && defer_small_group) { *defer_small_group = true; return cudaGetLastError(); }
    if (!small && d2moe_group_is_sortable(D.A, n_keys)) {
        const int threads = D.A >= 2048 ? 1024 : 512;
        const size_t gsm = group_sort_smem_ints(D.A, n_keys, threads / 32) * 4;
        cudaError_t e = ensure_dynamic_smem<&group_sort_kernel>((int)gsm);
        if (e != cudaSuccess) return e;
        launch_chained(group_sort_kernel, dim3(1), dim3(threads), gsm, st, D.A, n_keys, keys_ws, R.group_off, R.perm, R.inv_perm);
        return cudaGetLastError();
    }
    if (small || d2moe_group_is_mid(D.A, n_keys)) {
        const size_t gsm = (size_t)(((D.A + 31) & ~31) + n_keys + 1) * 4;
        cudaError_t e = ensure_dynamic_smem<&group_block_kernel>((int)gsm);
        if (e != cudaSuccess) return e;
        const int blocks = small ? 1 : (n_keys < 16 ? n_keys : 16);
        launch_chained(group_block_kernel, dim3(blocks), dim3(1024), gsm, st, D.A, n_keys, keys_ws, R.group_off, R.perm, R.inv_perm);
        return cudaGetLastError();
    }
    launch_chained(count_kernel, dim3((n_keys + 3) / 4), dim3(128), 0, st, D.A, n_keys, keys_ws, hist_ws);
    launch_chained(scan_kernel, dim3(1), dim3(32), 0, st, n_keys, hist_ws, R.group_off);
    launch_chained(scatter_kernel, dim3((n_keys + 3) / 4), dim3(128), 0, st, D.A, n_keys, keys_ws, R.group_off, R.perm, R.inv_perm);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// d2moe_route_static_scratch: the routing call for callers that cannot hand over a workspace.
//
// Its scratch (the per-assignment sort keys and the (expert, width) histogram that d2moe_route keeps
// in the caller's workspace) lives in one file-scope device array, so the call needs no allocation
// of any kind.  The array is part of the library image: every GPU that loads the library holds these
// bytes until the process exits.
// ------------------------------------------------------------------------------------------------
#include <mutex>

#define D2MOE_STATIC_SCRATCH_BYTES ((D2MOE_STATIC_MAX_ASSIGNMENTS + D2MOE_STATIC_MAX_KEYS) * 4)

static __device__ __align__(256) unsigned char g_route_scratch[D2MOE_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_addr[kMaxDevices] = {};   // device address of g_route_scratch, per device ordinal
}  // namespace

extern "C" d2moe_status d2moe_route_static_scratch(const d2moe_config* c, int64_t T, const void* x,
                                                   const void* gate_w, const float* logits, const void* bit_w,
                                                   const int8_t* forced, int32_t* topk_idx, float* topk_w,
                                                   int8_t* bit_idx, int32_t* perm, int32_t* inv_perm,
                                                   int32_t* group_off, int32_t* device_status, void* stream) {
    d2moe_status s = d2moe_check_config(c);
    if (s != D2MOE_OK) return s;
    if (T < 0) return D2MOE_ERR_SHAPE;
    // the fixed scratch bounds the problem: say so instead of overrunning it
    if (T * c->top_k > D2MOE_STATIC_MAX_ASSIGNMENTS || c->n_experts * c->n_bits > D2MOE_STATIC_MAX_KEYS)
        return D2MOE_ERR_WORKSPACE;
    if (!topk_idx || !topk_w || !bit_idx || !perm || !inv_perm || !group_off) return D2MOE_ERR_NULL;
    if (T > 0 && !x) return D2MOE_ERR_NULL;
    if ((gate_w == nullptr) == (logits == nullptr)) return D2MOE_ERR_NULL;
    if ((bit_w == nullptr) == (forced == nullptr)) return D2MOE_ERR_NULL;

    // In host code `g_route_scratch` is only a handle for the symbol, not an address a kernel can
    // use.  The device address is looked up once per device, with that device current, and kept.
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return D2MOE_ERR_CUDA;
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_scratch_mutex);
        if (!g_scratch_addr[dev]) {
            void* addr = nullptr;
            if (cudaGetSymbolAddress(&addr, g_route_scratch) != cudaSuccess || !addr) return D2MOE_ERR_CUDA;
            g_scratch_addr[dev] = addr;
        }
        scratch = g_scratch_addr[dev];
    }

    cudaStream_t st = (cudaStream_t)stream;
    const int n_keys = c->n_experts * c->n_bits;
    if (T == 0) {
        cudaError_t e = cudaMemsetAsync(group_off, 0, (size_t)(n_keys + 1) * 4, st);
        return e == cudaSuccess ? D2MOE_OK : D2MOE_ERR_CUDA;
    }
    MoeDims D;
    D.T = (int)T; D.d = c->d_model; D.F = c->d_ffn; D.E = c->n_experts; D.k = c->top_k;
    D.n_shared = c->n_shared; D.g = c->group_size; D.K = c->n_bits;
    for (int i = 0; i < 8; ++i) D.bits[i] = i < c->n_bits ? c->bits[i] : 0;
    D.A = (int)(T * c->top_k);
    D.A_tot = D.A + (int)(T * c->n_shared);
    D.renormalize = c->renormalize;
    // Nothing in the scratch has to start at zero: the key of every assignment and the count of every
    // (expert, width) pair are written before they are read, so the previous call's contents are inert.
    int32_t* keys = reinterpret_cast<int32_t*>(scratch);
    int32_t* hist = keys + D2MOE_STATIC_MAX_ASSIGNMENTS;
    RouteBufs R{topk_idx, topk_w, bit_idx, perm, inv_perm, group_off};
    launch_chain_begin();
    cudaError_t e = launch_route(D, (const __nv_bfloat16*)x, (const __nv_bfloat16*)gate_w, logits,
                                 (const __nv_bfloat16*)bit_w, forced, R, nullptr, keys, hist, device_status, st);
    return e == cudaSuccess ? D2MOE_OK : D2MOE_ERR_CUDA;
}
