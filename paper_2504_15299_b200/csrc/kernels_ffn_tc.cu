// Grouped dequant-GEMM on the 5th-generation tensor cores (tcgen05 + TMEM) for the expert FFN.
//
// One CTA computes, for one (unit, 128-row tile) pair, D[128 weight rows, N tokens] over a range of
// K-groups.  A "unit" is up to n_cap consecutive columns (tokens) of one expert in the padded,
// (expert, width)-sorted activation buffer; it holds one piece per routed width, each padded to a
// multiple of 16 columns.  Weight rows sit on the MMA's M side (TMEM lanes), tokens on N.
//
// Per K-group (g input columns) the four dequant warps own one weight row each (thread = row = TMEM
// lane).  A thread reads its row's packed segments from shared memory and builds the fp16 weights
// width by width, in registers, using the additivity of the nested code (Section 3.3.1,
// W_hat_{b_k} = W_hat_{b_1} + sum of the residual terms):
//     U_0  = (lo - s1/2) + s1 * v_0                       v_j = value of segment j
//     U_j  = U_{j-1} + M_j * v_j,   M_j = s1 / 2^(bits[j]-bits[0])
//     W_hat at width bits[j] = U_j + M_j / 2
// Each step is one AND (isolates a code pair inside the fp16 subnormal range, where a bit pattern
// v << p is the value v * 2^(p-24)) and one packed half-precision FMA with a pre-scaled multiplier.
// Every width that has tokens in the unit gets its tile written to TMEM (tcgen05.st) and one
// tcgen05.mma (A from TMEM, B = the tokens of that width from shared memory) accumulates it into
// the D columns of those tokens, so each packed byte is read once from HBM however many widths
// use it (the plane reuse of Section 3.4), and each token is multiplied exactly once.
// All tiles carry a common power-of-two factor 2^-S (S per matrix, from the largest scale seen at
// pack time) so that the multipliers stay inside fp16 range; the epilogue multiplies by 2^S.
//
// Warp roles (352 threads, 1 CTA per SM, all 512 TMEM columns): warps 0-3 and 4-7 are two dequant
// warpgroups, each owning one K-half of every tile (thread = weight row = TMEM lane; lanes 2i and 2i + 1
// hold row i of the tile's two packed blocks, for gate/up the two rows of one hidden unit, which the
// epilogue pairs with a shuffle) and taking alternate 16-column chunks of the epilogue; warp 8 streams packed blocks (cp.async.bulk), warp 9
// streams activation tiles (TMA, 128B swizzle, boxes of up to 256 rows), warp 10 issues the MMAs (the
// whole warp runs the loop, one elected lane issues).  A unit holds up to 320 tokens, so that one
// dequantization of a weight tile is amortised over enough tensor work to leave the kernel bound by
// the tensor cores; an MMA covers at most 256 of a piece's columns.  Work items (unit x tile) are taken
// from a global counter by the weight producer and published to the other warps through a queue in
// shared memory; the units are ordered by decreasing work.  Every wait is bounded: on expiry
// the CTA raises D2MOE_DEV_TIMEOUT, stops waiting, drains and exits.
#include "d2moe_common.cuh"
#include "kernels_ffn_tc.cuh"
#include "tc_common.cuh"

#include <type_traits>

namespace {

constexpr int TC_THREADS = 352;        // 8 dequant warps (2 warpgroups) + weight producer + activation producer + MMA issuer
constexpr int WARP_WPROD = 8, WARP_BPROD = 9, WARP_MMA = 10;
constexpr int TMEM_COLS = 512;
constexpr int D_COLS = 384;            // accumulator columns (n_cap <= 320)
constexpr int A_SLOTS = 2;             // operand tiles of GS/2 columns at TMEM columns 384 and 448
constexpr int NSB = 2;                 // activation ring depth
constexpr int MAX_NSW = 4;             // weight ring depth (upper bound)
constexpr int NSQ = 4;                 // entries of the work queue between the weight producer and the other warps

struct TcParams {
    MoeDims D;
    PackLayout L;
    ExpertPtrs P;
    int mode;                 // 0: gate/up + SwiGLU -> hbuf;  1: down -> obuf
    int n_cap, n_row_tiles, n_split, groups_per_split, nsw;
    const TcUnit* units;
    const int* n_units;
    int* next_item;           // work counter of this launch: starts at the grid size (item i < grid goes to CTA i)
    __half* hbuf;             // [R, F]
    float* obuf;              // [n_split][R, d]
    const float* row_scale;   // [3][R]: per padded row the power-of-two factors of the activation scaling (see tc_gather_kernel)
    long long R_alloc;
    int32_t* status;
    int smem_w_off, smem_bar_off;
};

// Packed half-precision arithmetic on raw 32-bit registers (a pair of halves each): the running tile lives in plain
// registers, so nothing is moved between a bit pattern and a half2 value.
__device__ __forceinline__ uint32_t hfma2_bits(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t hadd2_bits(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("add.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// ------------------------------------------------------------------------------------------------
// Dequantization of one K-half of one segment of one row into the running tile.
//   seg     shared-memory address of the segment inside the block (this row's chunks are at
//           (c*64 + rr)*cs)
//   half    which half of the group's g elements this warpgroup owns (0 or 1)
//   acc     running tile U (GS/4 half2 registers: register i = elements 2i, 2i+1 of the half)
//   m0      multiplier for a code at bit position 0: M_j * 2^(24 - S); position p uses m0 * 2^-p
//   FIRST   segment 0: the addend is u0 = (lo - s1/2) * 2^-S instead of acc
// ------------------------------------------------------------------------------------------------
template <int GS, int SW, bool FIRST>
__device__ __forceinline__ void dequant_segment(uint32_t seg, int rr, int half, uint32_t (&acc)[GS / 4], __half2 m0, __half2 u0) {
    constexpr int ROW_BYTES = GS * SW / 8;
    constexpr int CS = ROW_BYTES < 16 ? ROW_BYTES : 16;
    constexpr int HB = ROW_BYTES / 2;            // bytes of this half
    constexpr int LD = HB < 16 ? HB : 16;
    constexpr int NLD = HB / LD;
    constexpr int WPL = LD / 4;                 // words per load
    constexpr int PER = 16 / SW;                // registers per word
    constexpr int NPOS = 8 / SW;                // distinct bit positions per byte lane
    constexpr uint32_t FIELD = ((1u << SW) - 1u) * 0x00010001u;
    __half2 mult[NPOS];
    mult[0] = m0;
    const __half2 step = __float2half2_rn(1.0f / (float)(1 << SW));     // exact power of two
#pragma unroll
    for (int q = 1; q < NPOS; ++q) mult[q] = __hmul2(mult[q - 1], step);
#pragma unroll
    for (int l = 0; l < NLD; ++l) {
        uint32_t w[WPL];
        const int off = half * HB + l * LD;
        const int c = off / CS, within = off % CS;
        const uint32_t addr = seg + (uint32_t)((c * D2MOE_TILE_ROWS + rr) * CS + within);
        if constexpr (WPL == 4) {
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(addr));
        } else if constexpr (WPL == 2) {
            asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(w[0]), "=r"(w[1]) : "r"(addr));
        } else {
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w[0]) : "r"(addr));
        }
#pragma unroll
        for (int q = 0; q < WPL; ++q) {
            const uint32_t lo8 = w[q], hi8 = w[q] >> 8;
#pragma unroll
            for (int e = 0; e < PER; ++e) {
                const uint32_t src = (e & 1) ? hi8 : lo8;       // pair e of the word: bytes (0,2) or (1,3), bit SW*(e/2)
                const int i = (l * WPL + q) * PER + e;
                acc[i] = hfma2_bits(src & (FIELD << ((e >> 1) * SW)), as_u32(mult[e >> 1]), FIRST ? as_u32(u0) : acc[i]);
            }
        }
    }
}

// Free residual scales (scale_mode 1): a segment after the first adds W one-bit steps, each with its own scale, so
// its codes are folded in bit by bit: U += (2 s_l) bit_l for every step l of the segment (the constant - s_l of
// W_hat = ... + s_l (2 bit_l - 1) is added when the tile is written).  mb[pos]: multiplier of a bit at position pos
// of its byte lane, 2 s_l 2^(24 - S - pos) for the step that bit belongs to (0 for the unused bits of the field).
template <int GS, int SW>
__device__ __forceinline__ void dequant_segment_bits(uint32_t seg, int rr, int half, uint32_t (&acc)[GS / 4], int W,
                                                     const __half2 (&mb)[8]) {
    constexpr int ROW_BYTES = GS * SW / 8;
    constexpr int CS = ROW_BYTES < 16 ? ROW_BYTES : 16;
    constexpr int HB = ROW_BYTES / 2;
    constexpr int LD = HB < 16 ? HB : 16;
    constexpr int NLD = HB / LD;
    constexpr int WPL = LD / 4;
    constexpr int PER = 16 / SW;
#pragma unroll
    for (int l = 0; l < NLD; ++l) {
        uint32_t w[WPL];
        const int off = half * HB + l * LD;
        const int c = off / CS, within = off % CS;
        const uint32_t addr = seg + (uint32_t)((c * D2MOE_TILE_ROWS + rr) * CS + within);
        if constexpr (WPL == 4) {
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(addr));
        } else if constexpr (WPL == 2) {
            asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(w[0]), "=r"(w[1]) : "r"(addr));
        } else {
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w[0]) : "r"(addr));
        }
#pragma unroll
        for (int q = 0; q < WPL; ++q) {
            const uint32_t lo8 = w[q], hi8 = w[q] >> 8;
#pragma unroll
            for (int e = 0; e < PER; ++e) {
                const uint32_t src = (e & 1) ? hi8 : lo8;
                const int i = (l * WPL + q) * PER + e;
#pragma unroll
                for (int t = 0; t < SW; ++t) {
                    if (t < W) {
                        const int pos = (e >> 1) * SW + t;
                        acc[i] = hfma2_bits(src & (0x00010001u << pos), as_u32(mb[pos]), acc[i]);
                    }
                }
            }
        }
    }
}

template <int GS>
__device__ __forceinline__ void dequant_bits_dispatch(int sw, uint32_t seg, int rr, int half, uint32_t (&acc)[GS / 4], int W,
                                                      const __half2 (&mb)[8]) {
    switch (sw) {
        case 1: dequant_segment_bits<GS, 1>(seg, rr, half, acc, W, mb); break;
        case 2: dequant_segment_bits<GS, 2>(seg, rr, half, acc, W, mb); break;
        case 4: dequant_segment_bits<GS, 4>(seg, rr, half, acc, W, mb); break;
        default: dequant_segment_bits<GS, 8>(seg, rr, half, acc, W, mb); break;
    }
}

template <int GS, bool FIRST>
__device__ __forceinline__ void dequant_dispatch(int sw, uint32_t seg, int rr, int half, uint32_t (&acc)[GS / 4], __half2 m0, __half2 u0) {
    switch (sw) {
        case 1: dequant_segment<GS, 1, FIRST>(seg, rr, half, acc, m0, u0); break;
        case 2: dequant_segment<GS, 2, FIRST>(seg, rr, half, acc, m0, u0); break;
        case 4: dequant_segment<GS, 4, FIRST>(seg, rr, half, acc, m0, u0); break;
        default: dequant_segment<GS, 8, FIRST>(seg, rr, half, acc, m0, u0); break;
    }
}

struct ItemInfo {
    int unit, tile, split, g0, g1;
};

__device__ __forceinline__ ItemInfo decode_item(const TcParams& p, int item) {
    ItemInfo it;
    const int per_unit = p.n_row_tiles * p.n_split;
    it.unit = item / per_unit;
    const int rem = item - it.unit * per_unit;
    it.tile = rem / p.n_split;
    it.split = rem - it.tile * p.n_split;
    it.g0 = it.split * p.groups_per_split;
    it.g1 = min(p.L.n_groups, it.g0 + p.groups_per_split);
    return it;
}

// ------------------------------------------------------------------------------------------------
// The kernel
// ------------------------------------------------------------------------------------------------
template <int GS, int WPACK>
__global__ void __launch_bounds__(TC_THREADS, 1)
ffn_tc_kernel(const __grid_constant__ TcParams p, const __grid_constant__ TmaMaps maps) {
    constexpr int HALVES = GS / 64;              // 64-element K slabs of the activation tile
    constexpr int TILE_COLS = GS / 2;            // TMEM columns of one operand tile
    extern __shared__ uint8_t smem_raw[];
    // shared layout (from a 1024-byte boundary, which the 128B-swizzled operand tiles need):
    // [activation ring: NSB x n_cap*GS*2] [weight ring: nsw x 2 blocks] [barriers]
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t b_slot_bytes = (uint32_t)p.n_cap * GS * 2;
    const uint32_t w_slot_bytes = 2u * (uint32_t)p.L.block_bytes;
    const uint32_t bbuf = smem_base;
    const uint32_t wbuf = smem_base + p.smem_w_off;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.smem_bar_off);
    const uint32_t bar0 = smem_u32(bars);
    auto W_FULL = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    auto W_EMPTY = [&](int i) { return bar0 + 8u * (uint32_t)(MAX_NSW + i); };
    auto B_FULL = [&](int i) { return bar0 + 8u * (uint32_t)(2 * MAX_NSW + i); };
    auto B_EMPTY = [&](int i) { return bar0 + 8u * (uint32_t)(2 * MAX_NSW + NSB + i); };
    auto A_FULL = [&](int i) { return bar0 + 8u * (uint32_t)(2 * MAX_NSW + 2 * NSB + i); };
    auto A_EMPTY = [&](int i) { return bar0 + 8u * (uint32_t)(2 * MAX_NSW + 2 * NSB + A_SLOTS + i); };
    const uint32_t D_FULL = bar0 + 8u * (uint32_t)(2 * MAX_NSW + 2 * NSB + 2 * A_SLOTS);
    const uint32_t D_EMPTY = D_FULL + 8u;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * MAX_NSW + 2 * NSB + 2 * A_SLOTS + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    // Work queue (bytes 160..255 of the barrier block): the weight producer takes work items from a global
    // counter and publishes them to the other warps, so that CTAs that drew cheap items take more of them.
    // An entry is released by the activation producer, the issuer warp and the eight dequant warps.
    static_assert(8 * (2 * MAX_NSW + 2 * NSB + 2 * A_SLOTS + 2) + 8 <= 160, "barrier block");
    auto SQ_FULL = [&](uint32_t i) { return bar0 + 160u + 8u * i; };
    auto SQ_EMPTY = [&](uint32_t i) { return bar0 + 192u + 8u * i; };
    volatile int* sq_item = reinterpret_cast<volatile int*>(reinterpret_cast<uint8_t*>(bars) + 240);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < MAX_NSW; ++i) { mbar_init(W_FULL(i), 1); mbar_init(W_EMPTY(i), 256); }
        for (int i = 0; i < NSB; ++i) { mbar_init(B_FULL(i), 1); mbar_init(B_EMPTY(i), 1); }
        for (int i = 0; i < A_SLOTS; ++i) { mbar_init(A_FULL(i), 256); mbar_init(A_EMPTY(i), 1); }
        mbar_init(D_FULL, 1);
        mbar_init(D_EMPTY, 256);
        for (int i = 0; i < NSQ; ++i) { mbar_init(SQ_FULL(i), 1); mbar_init(SQ_EMPTY(i), 10); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // per-width constants of the dequant loop, read from shared memory instead of the kernel parameters
    // (a dynamically indexed parameter read costs a constant-cache round trip per tile)
    // per stored segment: {storage width | width index << 8 | last segment of its width << 16, byte offset,
    // bits of 2^(position - (top - b1)), scale_mode 1: byte offset of the scale of the field's lowest bit}
    int4* seg_tab = reinterpret_cast<int4*>(reinterpret_cast<uint8_t*>(bars) + 256);
    if (threadIdx.x < 8) {
        const int j = threadIdx.x;
        const int kk = p.L.seg_kk[j];
        const int last = (j < p.L.n_seg && p.L.last_seg[kk] == j) ? 1 : 0;
        const int e = p.L.seg_shift[j] - (p.L.top - p.L.b1);
        const int sc_t0 = p.L.w_sc_off[kk] + ((p.L.top - p.L.b1 - 1 - p.L.seg_shift[j]) - p.L.w_lv0[kk]) * D2MOE_TILE_ROWS * 2;
        seg_tab[j] = make_int4(p.L.seg_sw[j] | (kk << 8) | (last << 16), p.L.seg_off[j], (127 + e) << 23, sc_t0);
    }
    if (warp == WARP_MMA) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t d_tmem = tmem_base;                       // columns [0, n_cap)
    const uint32_t a_tmem = tmem_base + D_COLS;              // A_SLOTS tiles, 64 columns apart

    // set-up done (barriers, TMEM): from here on the kernel reads what the kernels before it wrote
    pdl_wait();
    const int n_units = *p.n_units;
    const int total_items = n_units * p.n_row_tiles * p.n_split;
    const int nsw = p.nsw;
    // next work item of a consumer: queue entry qi (one arrival per warp, or per thread for a single-thread role)
    auto pop = [&](uint32_t qi, bool whole_warp) -> int {
        const uint32_t q = qi & (NSQ - 1);
        mbar_wait(SQ_FULL(q), (qi / NSQ) & 1u, abort_flag, p.status);
        const int item = sq_item[q];
        if (whole_warp) __syncwarp();
        if (!whole_warp || lane == 0) mbar_arrive(SQ_EMPTY(q));
        return item;
    };

    if (warp == WARP_WPROD) {
        // ---------------- weight producer ----------------
        if (lane == 0) {
            uint32_t it = 0, wph = 0;
            int ws = 0;
            int item = blockIdx.x;
            for (uint32_t qi = 0;; ++qi) {
                const uint32_t q = qi & (NSQ - 1);
                mbar_wait(SQ_EMPTY(q), ((qi / NSQ) & 1u) ^ 1u, abort_flag, p.status);
                if (item >= total_items) item = -1;                    // the end mark
                sq_item[q] = item;
                mbar_arrive(SQ_FULL(q));
                if (item < 0) break;
                const int next = atomicAdd(p.next_item, 1);            // in flight while this item's blocks are issued
                const ItemInfo ii = decode_item(p, item);
                const TcUnit* u = p.units + ii.unit;
                const int e = u->e, kmax = u->kmax;
                const uint32_t bytes = (uint32_t)d2moe_prefix_bytes(p.L, kmax);
                const uint8_t *m0, *m1;
                int rt0, rt1;
                if (p.mode == 0) { m0 = p.P.w[3 * e + 0]; m1 = p.P.w[3 * e + 1]; rt0 = rt1 = ii.tile; }
                else { m0 = m1 = p.P.w[3 * e + 2]; rt0 = 2 * ii.tile; rt1 = 2 * ii.tile + 1; }
                for (int G = ii.g0; G < ii.g1; ++G, ++it) {
                    const int s = ws;                                  // ring slot and parity advance by addition
                    mbar_wait(W_EMPTY(s), wph ^ 1u, abort_flag, p.status);
                    if (++ws == nsw) { ws = 0; wph ^= 1u; }
                    mbar_expect_tx(W_FULL(s), 2 * bytes);
                    const uint32_t dst = wbuf + s * w_slot_bytes;
                    bulk_g2s(dst, m0 + d2moe_block_offset(p.L, rt0, G), bytes, W_FULL(s));
                    bulk_g2s(dst + p.L.block_bytes, m1 + d2moe_block_offset(p.L, rt1, G), bytes, W_FULL(s));
                }
                item = next;
            }
            // drain: every copy issued must have landed before the CTA may exit
            for (int s = 0; s < nsw && s < (int)it; ++s) {
                const uint32_t last = it - 1 - (it - 1 - s) % nsw;   // last iteration that used slot s
                mbar_wait(W_FULL(s), (last / nsw) & 1, abort_flag, p.status, true);
            }
        }
    } else if (warp == WARP_BPROD) {
        // ---------------- activation producer ----------------
        if (lane == 0) {
            uint32_t it = 0;
            for (uint32_t qi = 0;; ++qi) {
                const int item = pop(qi, false);
                if (item < 0) break;
                const ItemInfo ii = decode_item(p, item);
                const TcUnit* u = p.units + ii.unit;
                const int ncols = u->ncols;                       // multiple of 16, <= n_cap
                const int row0 = u->row0;                         // read once: the copies below are issued back to back
                const uint32_t bytes = (uint32_t)ncols * 128u * HALVES;
                for (int G = ii.g0; G < ii.g1; ++G, ++it) {
                    const int s = it % NSB;
                    mbar_wait(B_EMPTY(s), ((it / NSB) & 1) ^ 1, abort_flag, p.status);
                    mbar_expect_tx(B_FULL(s), bytes);
                    const uint32_t dst = bbuf + s * b_slot_bytes;
                    // the rows of the unit as boxes of 256, 128, 64, 32, 16 rows (largest first)
                    int r = 0;
                    for (int mi = 4; mi >= 0; --mi) {
                        const int box = 16 << mi;
                        while (ncols - r >= box) {
#pragma unroll
                            for (int h = 0; h < HALVES; ++h)
                                tma_load_2d(dst + h * (uint32_t)p.n_cap * 128u + (uint32_t)r * 128u, &maps.m[mi],
                                            G * GS + h * 64, row0 + r, B_FULL(s));
                            r += box;
                        }
                    }
                }
            }
            for (int s = 0; s < NSB && s < (int)it; ++s) {
                const uint32_t last = it - 1 - (it - 1 - s) % NSB;
                mbar_wait(B_FULL(s), (last / NSB) & 1, abort_flag, p.status, true);
            }
        }
    } else if (warp == WARP_MMA) {
        // ---------------- MMA issuer (whole warp runs the loop, one elected lane issues) ----------------
        // The issuer is a serial resource (one hand-off per tile), so everything an MMA needs is a register
        // add away: per item the pieces' instruction descriptors, D columns and row offsets (an MMA covers at
        // most 256 columns: a piece is at most two chunks); per stage the low word of the shared-memory
        // descriptor (its high word is a constant).
        constexpr uint32_t DESC_HI = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);
        uint32_t it = 0, at = 0, ic = 0;
        const uint32_t slab_step = (uint32_t)p.n_cap * 8u;        // second 64-column slab of a stage, in 16-byte units
        for (uint32_t qi = 0;; ++qi, ++ic) {
            const int item = pop(qi, true);
            if (item < 0) break;
            const ItemInfo ii = decode_item(p, item);
            const TcUnit* u = p.units + ii.unit;
            const int kmax = u->kmax;
            uint32_t id0[8], id1[8], dc[8], bo[8];                // chunk 0 / chunk 1 descriptors, D column, B rows / 16 B
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const int cnt = kk <= kmax ? u->cnt[kk] : 0;
                const int col0 = u->col0[kk];
                id0[kk] = cnt ? instr_desc_f16(min(cnt, 256)) : 0u;
                id1[kk] = cnt > 256 ? instr_desc_f16(cnt - 256) : 0u;
                dc[kk] = d_tmem + col0;
                bo[kk] = (uint32_t)col0 * 8u;
            }
            mbar_wait(D_EMPTY, (ic & 1) ^ 1, abort_flag, p.status);
            tc_fence_after();
            for (int G = ii.g0; G < ii.g1; ++G, ++it) {
                const int s = it % NSB;
                mbar_wait(B_FULL(s), (it / NSB) & 1, abort_flag, p.status);
                const uint32_t blo = (((bbuf + s * b_slot_bytes) & 0x3FFFFu) >> 4) | (1u << 16);
                const uint32_t accum = (G != ii.g0) ? 1u : 0u;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    if (id0[kk] == 0u) continue;
                    const uint32_t slot = at & 1u;
                    mbar_wait(A_FULL(slot), (at >> 1) & 1u, abort_flag, p.status);
                    tc_fence_after();
                    if (elect_one()) {
                        const uint32_t a_addr = a_tmem + slot * 64;
                        const uint32_t lo = blo + bo[kk];
#pragma unroll
                        for (int j = 0; j < GS / 16; ++j)
                            tc_mma_ts_lohi(dc[kk], a_addr + j * 8, lo + (j >> 2) * slab_step + (j & 3) * 2, DESC_HI, id0[kk],
                                           j == 0 ? accum : 1u);
                        if (id1[kk] != 0u) {
#pragma unroll
                            for (int j = 0; j < GS / 16; ++j)
                                tc_mma_ts_lohi(dc[kk] + 256, a_addr + j * 8, lo + 256 * 8 + (j >> 2) * slab_step + (j & 3) * 2, DESC_HI,
                                               id1[kk], j == 0 ? accum : 1u);
                        }
                        tc_commit(A_EMPTY(slot));
                    }
                    __syncwarp();
                    ++at;
                }
                if (elect_one()) tc_commit(B_EMPTY(s));
                __syncwarp();
            }
            if (elect_one()) tc_commit(D_FULL);
            __syncwarp();
        }
        // all MMAs must be complete before TMEM is freed
        if (ic > 0) mbar_wait(D_FULL, (ic - 1) & 1, abort_flag, p.status, true);
    } else {
        // ---------------- dequant + epilogue warps: warpgroup wg owns K-half wg of every tile ----------------
        const int wg = warp >> 2;
        const int r = threadIdx.x & 127;         // row of the tile = TMEM lane
        // lanes 2i and 2i + 1 hold row i of the tile's first and second packed block (mode 0: the gate and the up row of
        // one hidden unit, which the epilogue pairs with a shuffle)
        const int blk = r & 1, rr = r >> 1;
        const uint32_t lane_addr = ((uint32_t)((warp & 3) * 32)) << 16;
        uint32_t it = 0, at = 0, ic = 0;
        uint32_t wph = 0;                               // weight ring: slot and parity advance by addition
        int ws = 0;
        uint32_t acc[GS / 4];                           // the running tile: packed half pairs
        for (uint32_t qi = 0;; ++qi, ++ic) {
            const int item = pop(qi, true);
            if (item < 0) break;
            const ItemInfo ii = decode_item(p, item);
            const TcUnit* u = p.units + ii.unit;
            const int e = u->e, kmax = u->kmax;
            const uint8_t* mat = p.mode == 0 ? p.P.w[3 * e + blk] : p.P.w[3 * e + 2];
            const int S = matrix_exponent(mat);
            const float two_mS = exp2f((float)-S);
            unsigned present = 0;
            for (int kk = 0; kk <= kmax; ++kk) present |= (u->cnt[kk] > 0 ? 1u : 0u) << kk;
            const long long row0 = u->row0;                      // read here: the epilogue must not wait for it
            const int ncols = u->ncols;

#pragma unroll 1
            for (int G = ii.g0; G < ii.g1; ++G, ++it) {
                const int s = ws;
                mbar_wait(W_FULL(s), wph, abort_flag, p.status);
                if (++ws == nsw) { ws = 0; wph ^= 1u; }
                const uint32_t wb = wbuf + s * w_slot_bytes + blk * p.L.block_bytes;
                uint32_t meta;
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(meta) : "r"(wb + 4u * rr));
                const __half2 mh = as_h2(meta);
                const float s1 = __low2float(mh), lo = __high2float(mh);
                const __half2 u0 = h2dup((lo - 0.5f * s1) * two_mS);
                // hands the running tile over as the tile of a width index; addend: what the tile lacks of W_hat 2^-S
                // (tied scales: half a step of that width, M_kk / 2)
                auto write_tile = [&](float addend) {
                    const int slot = at % A_SLOTS;
                    mbar_wait(A_EMPTY(slot), ((at / A_SLOTS) & 1) ^ 1, abort_flag, p.status);
                    tc_fence_after();
                    const __half2 half_m = h2dup(addend);
                    const uint32_t dst = a_tmem + slot * 64 + wg * (TILE_COLS / 2) + lane_addr;
#pragma unroll
                    for (int c = 0; c < GS / 64; ++c) {
#pragma unroll
                        for (int h8 = 0; h8 < 2; ++h8) {
                            uint32_t v[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) v[j] = hadd2_bits(acc[c * 16 + h8 * 8 + j], as_u32(half_m));
                            tc_st8(dst + c * 16 + h8 * 8, v);
                        }
                    }
                    tc_wait_st();
                    tc_fence_before();
                    mbar_arrive(A_FULL(slot));
                    ++at;
                };
                if constexpr (WPACK != 0) {
                    // compile-time width list: storage widths, segment offsets and scale ratios are immediates
                    using WL = WidthList<WPACK>;
                    auto seg_step = [&](auto jc) {
                        constexpr int J = decltype(jc)::value;
                        if constexpr (J < WL::count()) {
                            if (J <= kmax) {
                                constexpr int db = WL::top() - WL::pos(J) - WL::w(0);      // bits[J] - bits[0]
                                const float Mk = s1 * __int_as_float((127 - db) << 23) * two_mS;
                                dequant_segment<GS, WL::sw(J), J == 0>(wb + (uint32_t)WL::seg_off(GS, J), rr, wg, acc,
                                                                      h2dup(Mk * 16777216.0f), u0);
                                if ((present >> J) & 1u) write_tile(0.5f * Mk);
                            }
                        }
                    };
                    // free residual scales: W_hat = lo + s1 Q + sum over the steps of s_l (2 bit_l - 1); a step's w one-bit
                    // levels each bring their own scale (stored in front of the step's codes)
                    float cneg = 0.0f;                           // - sum of the scales folded in so far, times 2^-S
                    auto seg_step_free = [&](auto jc) {
                        constexpr int J = decltype(jc)::value;
                        if constexpr (J < WL::count()) {
                            if (J <= kmax) {
                                const uint32_t seg = wb + (uint32_t)p.L.seg_off[J];
                                if constexpr (J == 0) {
                                    dequant_segment<GS, WL::sw(0), true>(seg, rr, wg, acc, h2dup(s1 * two_mS * 16777216.0f),
                                                                         h2dup(lo * two_mS));
                                } else {
                                    constexpr int SW = WL::sw(J);
                                    // this row's scale of the field's lowest bit; bit t of the field: t planes before
                                    const uint32_t sc = wb + (uint32_t)(p.L.w_sc_off[J] + ((p.L.top - p.L.b1 - 1 - p.L.seg_shift[J]) - p.L.w_lv0[J]) * D2MOE_TILE_ROWS * 2)
                                                      + 2u * rr;
                                    float sl2[SW];
#pragma unroll
                                    for (int t = 0; t < SW; ++t) {
                                        unsigned short raw;
                                        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(raw) : "r"(sc - (uint32_t)(t * D2MOE_TILE_ROWS * 2)));
                                        const float sl = __half2float(__ushort_as_half(raw)) * two_mS;
                                        cneg -= sl;
                                        sl2[t] = 2.0f * sl;
                                    }
                                    __half2 mb[8];
#pragma unroll
                                    for (int pos = 0; pos < 8; ++pos)
                                        mb[pos] = h2dup(sl2[pos % SW] * __int_as_float((127 + 24 - pos) << 23));
                                    dequant_segment_bits<GS, SW>(seg, rr, wg, acc, SW, mb);
                                }
                                if ((present >> J) & 1u) write_tile(cneg);
                            }
                        }
                    };
                    if (p.L.scale_mode == 1) {
                        seg_step_free(std::integral_constant<int, 0>{});
                        seg_step_free(std::integral_constant<int, 1>{});
                        seg_step_free(std::integral_constant<int, 2>{});
                        seg_step_free(std::integral_constant<int, 3>{});
                    } else {
                        seg_step(std::integral_constant<int, 0>{});
                        seg_step(std::integral_constant<int, 1>{});
                        seg_step(std::integral_constant<int, 2>{});
                        seg_step(std::integral_constant<int, 3>{});
                    }
                } else {
                    const int smax = p.L.last_seg[kmax];         // stored segments 0..smax
                    if (p.L.scale_mode == 1) {
                        // free residual scales: W_hat = lo + s1 Q + sum over the steps of s_l (2 bit_l - 1)
                        float cneg = 0.0f;                       // - sum of the scales of the steps folded in so far, times 2^-S
#pragma unroll 1
                        for (int sj = 0; sj <= smax; ++sj) {
                            const int4 tb = seg_tab[sj];
                            const int sw = tb.x & 255, kk = (tb.x >> 8) & 255;
                            const uint32_t seg = wb + (uint32_t)tb.y;
                            if (kk == 0) {                       // a field of the base code: s1 times its value at its position
                                const __half2 m0 = h2dup(s1 * __int_as_float(tb.z) * two_mS * 16777216.0f);
                                if (sj == 0) dequant_dispatch<GS, true>(sw, seg, rr, wg, acc, m0, h2dup(lo * two_mS));
                                else dequant_dispatch<GS, false>(sw, seg, rr, wg, acc, m0, u0);
                            } else {
                                const uint32_t sc = wb + (uint32_t)tb.w + 2u * rr;       // this row's scale of the field's lowest bit
                                // bit t of the field belongs to the step whose scale lies t planes before; the byte lane
                                // holds 8 / sw fields, so position pos carries the scale of bit pos % sw
                                float sl2[8];
#pragma unroll
                                for (int t = 0; t < 8; ++t) {
                                    sl2[t] = 0.0f;
                                    if (t < sw) {
                                        unsigned short raw;
                                        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(raw) : "r"(sc - (uint32_t)(t * D2MOE_TILE_ROWS * 2)));
                                        const float sl = __half2float(__ushort_as_half(raw)) * two_mS;
                                        cneg -= sl;                       // each step once
                                        sl2[t] = 2.0f * sl;
                                    }
                                }
                                __half2 mb[8];
#pragma unroll
                                for (int pos = 0; pos < 8; ++pos)
                                    mb[pos] = h2dup(sl2[pos & (sw - 1)] * __int_as_float((127 + 24 - pos) << 23));
                                dequant_bits_dispatch<GS>(sw, seg, rr, wg, acc, sw, mb);
                            }
                            if (((tb.x >> 16) & 1) && ((present >> kk) & 1u)) write_tile(cneg);
                        }
                    } else {
#pragma unroll 1
                        for (int sj = 0; sj <= smax; ++sj) {
                            const int4 tb = seg_tab[sj];
                            const int sw = tb.x & 255, kk = (tb.x >> 8) & 255;
                            // the field's multiplier: s1 2^(position - (top - b1)) 2^-S, and for a code at bit position 0 of its lane
                            const float Ms = s1 * __int_as_float(tb.z) * two_mS;
                            const __half2 m0 = h2dup(Ms * 16777216.0f);
                            const uint32_t seg = wb + (uint32_t)tb.y;
                            if (sj == 0) dequant_dispatch<GS, true>(sw, seg, rr, wg, acc, m0, u0);
                            else dequant_dispatch<GS, false>(sw, seg, rr, wg, acc, m0, u0);
                            // the last field of a width's step sits at that width's unit: half a step completes the tile
                            if (((tb.x >> 16) & 1) && ((present >> kk) & 1u)) write_tile(0.5f * Ms);
                        }
                    }
                }
                mbar_arrive(W_EMPTY(s));
            }

            // ---- epilogue: D (128 rows x ncols) -> global; the two warpgroups take alternate 16-column chunks ----
            // While it runs the tensor pipe is idle, so it is kept short: a warp finishes two chunks at a time (two
            // independent chains of tensor-memory load, shuffle, SwiGLU and stores), their scale factors are fetched a
            // pair ahead, and SwiGLU is split between the two threads of a hidden unit (the gate row's thread
            // finishes the first eight tokens of a chunk, the up row's thread the other eight).  Padding columns
            // (their activation rows and scale factors are never written) are neither stored nor checked.
            int pc0[8], pcn[8], prl[8];                          // per piece: first column, columns, real columns
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                pc0[kk] = u->col0[kk]; pcn[kk] = kk <= kmax ? u->cnt[kk] : 0; prl[kk] = u->real[kk];
            }
            auto nreal_of = [&](int c0) -> int {               // real tokens among the 16 columns from c0
                int nreal = 0;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const int rel = c0 - pc0[kk];
                    if (pcn[kk] > 0 && rel >= 0 && rel < pcn[kk]) nreal = min(16, max(0, prl[kk] - rel));
                }
                return nreal;
            };
            mbar_wait(D_FULL, ic & 1, abort_flag, p.status);
            tc_fence_after();
            const float two_S = exp2f((float)S);
            const int keep = blk == 0 ? 0 : 8;
            // mode 0: xs of the eight tokens this thread finishes, then hq of the same; mode 1: hs of all sixteen
            auto load_scales = [&](int c0, float4 (&sc)[4]) {
                const long long grow = row0 + c0;
                if (p.mode == 0) {
                    const float4* a = reinterpret_cast<const float4*>(p.row_scale + grow + keep);
                    const float4* b = reinterpret_cast<const float4*>(p.row_scale + p.R_alloc + grow + keep);
                    sc[0] = a[0]; sc[1] = a[1]; sc[2] = b[0]; sc[3] = b[1];
                } else {
                    const float4* a = reinterpret_cast<const float4*>(p.row_scale + 2 * p.R_alloc + grow);
                    sc[0] = a[0]; sc[1] = a[1]; sc[2] = a[2]; sc[3] = a[3];
                }
            };
            uint32_t overbits = 0;                               // largest |h| seen, as bits (a NaN above every number)
            auto finish = [&](int c0, const uint32_t (&v)[16], const float4 (&sc)[4]) {
                const long long grow = row0 + c0;
                const int nreal = nreal_of(c0);
                if (p.mode == 0) {
                    const float xs[8] = {sc[0].x, sc[0].y, sc[0].z, sc[0].w, sc[1].x, sc[1].y, sc[1].z, sc[1].w};
                    const float hq[8] = {sc[2].x, sc[2].y, sc[2].z, sc[2].w, sc[3].x, sc[3].y, sc[3].z, sc[3].w};
                    // exchange with the neighbouring lane (the other row of the hidden unit): the gate thread hands
                    // over tokens 8..15, the up thread tokens 0..7, already times their own matrix's 2^S
                    float other_v[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        other_v[j] = __shfl_xor_sync(0xffffffffu, __uint_as_float(blk == 0 ? v[8 + j] : v[j]) * two_S, 1);
                    __half* dst = p.hbuf + (grow + keep) * p.D.F + (long long)ii.tile * 64 + rr;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float mine = __uint_as_float(blk == 0 ? v[j] : v[8 + j]) * two_S * xs[j];
                        const float other = other_v[j] * xs[j];
                        const float g = blk == 0 ? mine : other, up = blk == 0 ? other : mine;
                        float h = __fdividef(g, 1.0f + __expf(-g)) * up * hq[j];
                        if (keep + j < nreal) {
                            const uint32_t hb = __float_as_uint(h) & 0x7fffffffu;
                            overbits = max(overbits, hb);
                            // beyond fp16 even at the token's own scale (or not a number): stored as zero, call flagged below
                            if (hb > 0x477fe000u) h = 0.0f;                  // bits of 65504
                            dst[(long long)j * p.D.F] = __float2half_rn(h);
                        }
                    }
                } else {
                    const float hs[16] = {sc[0].x, sc[0].y, sc[0].z, sc[0].w, sc[1].x, sc[1].y, sc[1].z, sc[1].w,
                                          sc[2].x, sc[2].y, sc[2].z, sc[2].w, sc[3].x, sc[3].y, sc[3].z, sc[3].w};
                    float* dst = p.obuf + (long long)ii.split * p.R_alloc * p.D.d + grow * p.D.d + (long long)ii.tile * 128 + blk * 64 + rr;
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (j < nreal) dst[(long long)j * p.D.d] = __uint_as_float(v[j]) * two_S * hs[j];
                }
            };
            float4 sa_next[4], sb_next[4];
            if (wg * 16 < ncols) load_scales(wg * 16, sa_next);
            if (wg * 16 + 32 < ncols) load_scales(wg * 16 + 32, sb_next);
            for (int c0 = wg * 16; c0 < ncols; c0 += 64) {
                const bool two = c0 + 32 < ncols;
                uint32_t va[16], vb[16];
                tc_ld16(d_tmem + lane_addr + c0, va);
                if (two) tc_ld16(d_tmem + lane_addr + c0 + 32, vb);
                float4 sa[4], sb[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) { sa[q] = sa_next[q]; sb[q] = sb_next[q]; }
                if (c0 + 64 < ncols) load_scales(c0 + 64, sa_next);
                if (c0 + 96 < ncols) load_scales(c0 + 96, sb_next);
                tc_wait_ld();
                finish(c0, va, sa);
                if (two) finish(c0 + 32, vb, sb);
            }
            if (p.mode == 0 && overbits > 0x477fe000u && p.status) atomicOr(p.status, D2MOE_DEV_NONFINITE);
            tc_fence_before();
            mbar_arrive(D_EMPTY);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == WARP_MMA) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------
// Unit construction and activation gather
// ------------------------------------------------------------------------------------------------
// One block.  Pads every (expert, width) group to a multiple of 16 rows, lays the groups out
// contiguously (routed experts, then shared experts), cuts each expert's range into units of at
// most n_cap rows, and records for every assignment its padded row.
__global__ void __launch_bounds__(256)
tc_prep_kernel(MoeDims D, RouteBufs R, int n_cap, TcUnit* units, int* n_units, int32_t* pad_off,
               int32_t* row_map, int32_t* src_token, int max_units, int ffn_grid, int32_t* status) {
    pdl_enter();
    __shared__ int s_total_rows, s_n_units;
    __shared__ int s_cost[1024];
    const int n_keys = D.E * D.K + D.n_shared;
    // 1. padded offsets (one warp scans)
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        int carry = 0;
        for (int base = 0; base < n_keys; base += 32) {
            const int i = base + lane;
            int n = 0;
            if (i < D.E * D.K) n = R.group_off[i + 1] - R.group_off[i];
            else if (i < n_keys) n = D.T;
            const int v = (n + 15) & ~15;
            int incl = v;
            for (int off = 1; off < 32; off <<= 1) {
                const int o = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += o;
            }
            if (i < n_keys) pad_off[i] = carry + incl - v;
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) { pad_off[n_keys] = carry; s_total_rows = carry; }
    }
    __syncthreads();
    const int total_rows = s_total_rows;
    // 2. source token of every padded row (-1 = padding)
    for (int i = threadIdx.x; i < total_rows; i += blockDim.x) src_token[i] = -1;
    __syncthreads();
    for (int a = threadIdx.x; a < D.A; a += blockDim.x) {
        const int pos = R.inv_perm[a];
        const int e = R.topk_idx[a], kk = R.bit_idx[a];
        // a supplied routing index out of range, or a position outside the group of (e, kk): the assignment is
        // skipped (row -1 contributes nothing to the combine) and the call is flagged
        const int key = e * D.K + kk;
        if (e < 0 || e >= D.E || kk < 0 || kk >= D.K || pos < R.group_off[key] || pos >= R.group_off[key + 1]) {
            row_map[a] = -1;
            if (status) atomicOr(status, D2MOE_DEV_BAD_INDEX);
            continue;
        }
        const int row = pad_off[key] + (pos - R.group_off[key]);
        row_map[a] = row;
        src_token[row] = a / D.k;
    }
    for (int i = threadIdx.x; i < D.n_shared * D.T; i += blockDim.x) {
        const int s = i / D.T, t = i - s * D.T;
        const int row = pad_off[D.E * D.K + s] + t;
        row_map[D.A + i] = row;
        src_token[row] = t;
    }
    // 3. units: a warp scans the experts' unit counts, then one thread per expert writes that expert's units
    __shared__ int s_uoff[D2MOE_MAX_EXPERTS + 1];
    const int n_exp = D.E + D.n_shared;
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        int carry = 0;
        for (int base = 0; base < n_exp; base += 32) {
            const int e = base + lane;
            int nu_e = 0;
            if (e < n_exp) {
                const int key0 = e < D.E ? e * D.K : D.E * D.K + (e - D.E);
                const int key1 = e < D.E ? key0 + D.K : key0 + 1;
                nu_e = (pad_off[key1] - pad_off[key0] + n_cap - 1) / n_cap;
            }
            int incl = nu_e;
            for (int off = 1; off < 32; off <<= 1) {
                const int o = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += o;
            }
            if (e < n_exp) s_uoff[e] = carry + incl - nu_e;
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) {
            const int nu = min(carry, max_units);
            s_uoff[n_exp] = carry;
            n_units[0] = nu;
            n_units[1] = ffn_grid; n_units[2] = ffn_grid;      // work counters of the two expert kernels
            s_n_units = nu;
        }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < n_exp; e += blockDim.x) {
        const int key0 = e < D.E ? e * D.K : D.E * D.K + (e - D.E);
        const int key1 = e < D.E ? key0 + D.K : key0 + 1;
        const int p0 = pad_off[key0], p1 = pad_off[key1];
        int nu = s_uoff[e];
        for (int start = p0; start < p1 && nu < max_units; start += n_cap, ++nu) {
            const int end = min(p1, start + n_cap);
            TcUnit u;
            u.e = e; u.row0 = start; u.ncols = end - start; u.kmax = 0;
            for (int kk = 0; kk < 8; ++kk) { u.col0[kk] = 0; u.cnt[kk] = 0; u.real[kk] = 0; }
            for (int key = key0; key < key1; ++key) {
                const int kk = e < D.E ? key - key0 : D.K - 1;
                const int a0 = pad_off[key], a1 = pad_off[key + 1];
                const int n_real = e < D.E ? R.group_off[key + 1] - R.group_off[key] : D.T;
                const int lo = max(a0, start), hi = min(a1, end);
                if (hi <= lo) continue;
                u.col0[kk] = lo - start;
                u.cnt[kk] = hi - lo;
                u.real[kk] = max(0, min(hi, a0 + n_real) - lo);
                u.kmax = kk;
            }
            // work per group: one dequantised tile per width present + tensor time per column
            int n_present = 0;
            for (int kk = 0; kk < 8; ++kk) n_present += u.cnt[kk] > 0 ? 1 : 0;
            if (nu < 1024) s_cost[nu] = 190 * n_present + u.ncols;
            units[nu] = u;
        }
    }
    __syncthreads();
    // 4. order the units by decreasing work, so that the expert kernels, whose CTAs draw work items from a
    //    counter, take the cheap ones last (rank by cost, ties by index; then permute)
    const int n = s_n_units;
    if (n <= 1024) {
        TcUnit mine[4];
        int rank[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int i = threadIdx.x + k * blockDim.x;
            rank[k] = -1;
            if (i < n) {
                mine[k] = units[i];
                const int c = s_cost[i];
                int rk = 0;
                for (int j = 0; j < n; ++j) rk += (s_cost[j] > c || (s_cost[j] == c && j < i)) ? 1 : 0;
                rank[k] = rk;
            }
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (rank[k] >= 0) units[rank[k]] = mine[k];
    }
}

// xp16[row, :] = fp16(x[src_token[row], :] * 2^(4-e)) for the real rows, where 2^e is the power of two just
// above the row's largest magnitude: every row enters the fp16 products with its largest element in
// [8, 16), whatever its own magnitude (a token of magnitude 1e5 or 1e-6 loses nothing to the fp16
// range).  row_scale[0][row] = 2^(e-4) undoes that in the gate/up epilogue; h = silu(g) * u grows like
// the square of the row's magnitude, so it is stored as fp16(h * row_scale[1][row]) with
// row_scale[1] = 2^-eh, eh = 2 (e - 4) (clamped to +-60), and the down projection's epilogue multiplies
// by row_scale[2] = 2^eh.  A row that holds a NaN or an infinity becomes zeros (scale 0: its outputs
// are zero) and the call is flagged.  Padding rows are never consumed: a D column depends only on its
// own token row.
__global__ void __launch_bounds__(128)
tc_gather_kernel(int d, const __nv_bfloat16* __restrict__ x, const int32_t* __restrict__ src_token,
                 const int32_t* __restrict__ pad_off, int n_keys, __half* __restrict__ xp16,
                 float* __restrict__ row_scale, long long R_alloc, int32_t* status) {
    pdl_enter();
    __shared__ float s_red[4];
    const int total_rows = pad_off[n_keys];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int row = blockIdx.x; row < total_rows; row += gridDim.x) {
        const int t = src_token[row];
        if (t < 0) continue;
        // eight elements (16 bytes) per thread and step; d is a multiple of 128 on this path
        const uint4* src = reinterpret_cast<const uint4*>(x + (size_t)t * d);
        uint4* dst = reinterpret_cast<uint4*>(xp16 + (size_t)row * d);
        float amax = 0.0f;
        int bad = 0;
        for (int i = threadIdx.x; i < d / 8; i += blockDim.x) {
            const uint4 v = src[i];
            const uint32_t* vi = reinterpret_cast<const uint32_t*>(&v);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&vi[k]));
                amax = fmaxf(amax, fmaxf(fabsf(f.x), fabsf(f.y)));
                bad |= !(fabsf(f.x) < 3.0e38f) | !(fabsf(f.y) < 3.0e38f);
            }
        }
        for (int off = 16; off; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
        bad = __syncthreads_or(bad);
        if (lane == 0) s_red[warp] = amax;
        __syncthreads();
        amax = fmaxf(fmaxf(s_red[0], s_red[1]), fmaxf(s_red[2], s_red[3]));
        __syncthreads();
        int e = 4;
        if (amax > 0.0f && !bad) frexpf(amax, &e);                   // amax = m 2^e, 0.5 <= m < 1
        const float mult = bad ? 0.0f : exp2f((float)(4 - e));
        if (threadIdx.x == 0) {
            const int eh = max(-60, min(60, 2 * (e - 4)));
            row_scale[row] = bad ? 0.0f : exp2f((float)(e - 4));
            row_scale[R_alloc + row] = exp2f((float)-eh);
            row_scale[2 * R_alloc + row] = exp2f((float)eh);
            if (bad && status) atomicOr(status, D2MOE_DEV_NONFINITE);
        }
        for (int i = threadIdx.x; i < d / 8; i += blockDim.x) {
            const uint4 v = src[i];
            uint4 o;
            const uint32_t* vi = reinterpret_cast<const uint32_t*>(&v);
            uint32_t* oi = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&vi[k]));
                const __half2 h = bad ? __floats2half2_rn(0.0f, 0.0f) : __floats2half2_rn(f.x * mult, f.y * mult);
                oi[k] = *reinterpret_cast<const uint32_t*>(&h);
            }
            dst[i] = o;
        }
    }
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
bool tc_path_supported(const d2moe_config* c) {
    if (c->group_size != 64 && c->group_size != 128) return false;
    if (c->d_ffn % 64 || c->d_model % 128) return false;
    return true;
}

void tc_plan(const d2moe_config* c, long long T, TcPlan* pl) {
    const long long A = T * c->top_k, A_tot = A + T * c->n_shared;
    const long long avg = (A + c->n_experts - 1) / c->n_experts;
    // up to about 40 tokens per expert the 8-bit kernel (units of 32 slots, weights unpacked once per unit) is
    // faster than the fp16 grouped GEMM (measured crossover on the Mixtral shape: T = 160, 40 tokens per expert)
    // (the 8-bit kernel folds one scale per group into its integer accumulators, which needs the tied residual
    // scales: with free scales every load takes the grouped GEMM)
    pl->decode = (avg <= D2MOE_DECODE_MAX_AVG && c->scale_mode == 0) ? 1 : 0;
    if (pl->decode) {
        pl->n_cap = 32;                      // token slots per unit
    } else {
        pl->n_cap = 320;
    }
    const long long n_pieces = pl->decode ? (long long)c->n_experts + c->n_shared
                                          : (long long)c->n_experts * c->n_bits + c->n_shared;
    // decode: every (expert, width) class is padded to 8 slots; otherwise pieces are padded to 16 rows
    const long long n_classes = (long long)c->n_experts * c->n_bits + c->n_shared;
    long long pad_rows = pl->decode ? A_tot + 7 * (n_classes < A_tot ? n_classes : A_tot)
                                    : A_tot + 15 * (n_pieces < A_tot ? n_pieces : A_tot);
    pl->R_alloc = ((pad_rows + 255) / 256) * 256 + 256;
    pl->max_units = (int)(c->n_experts + c->n_shared + pl->R_alloc / pl->n_cap + 1);
    // split-K of the down projection: aim for >= 4 work items per resident CTA
    long long units_est = (c->n_experts < A ? c->n_experts : A) + (long long)c->n_shared * ((T + pl->n_cap - 1) / pl->n_cap);
    // prefill-sized loads: an expert spans several units (every partial output plane is written by the down
    // projection and read again by the combine, so no more planes than the work distribution needs)
    if (!pl->decode && units_est < A / pl->n_cap + c->n_experts / 2) units_est = A / pl->n_cap + c->n_experts / 2;
    const long long tiles = c->d_model / 128;
    const int n_groups = c->d_ffn / c->group_size;
    const long long ctas = pl->decode ? 296 : 148;       // resident CTAs: 2 per SM (decode kernel), 1 per SM
    long long want = (4 * ctas + units_est * tiles - 1) / (units_est * tiles);
    if (want < 1) want = 1;
    if (want > 8) want = 8;
    if (want > n_groups / 4) want = n_groups / 4 > 0 ? n_groups / 4 : 1;
    // equal parts balance best: the largest divisor of the number of groups up to the wanted factor, unless
    // that halves it
    for (long long w = want; 2 * w > want; --w)
        if (n_groups % w == 0) { want = w; break; }
    pl->groups_per_split = (int)((n_groups + want - 1) / want);
    if (c->group_size == 64 && (pl->groups_per_split & 1)) ++pl->groups_per_split;   // whole 128-column ring stages
    pl->n_split = (n_groups + pl->groups_per_split - 1) / pl->groups_per_split;
}

cudaError_t launch_ffn_tensor(const d2moe_config* c, const MoeDims& D, const PackLayout& Lgu, const PackLayout& Ld,
                              const ExpertPtrs& P, const __nv_bfloat16* x, const RouteBufs& R, const TcPlan& pl,
                              const TcBuffers& B, int32_t* device_status, cudaStream_t st, void* const* ev) {
    auto mark = [&](int i) { if (ev) cudaEventRecord((cudaEvent_t)ev[i], st); };
    const int n_keys = D.E * D.K + D.n_shared;
    const int sms = device_sm_count();
    launch_chained(tc_prep_kernel, dim3(1), dim3(256), 0, st, D, R, pl.n_cap, B.units, B.n_units, B.pad_off, B.row_map, B.src_token, pl.max_units, sms,
                                      device_status);
    launch_chained(tc_gather_kernel, dim3(1184), dim3(128), 0, st, D.d, x, B.src_token, B.pad_off, n_keys, B.xp16, B.slot_f, pl.R_alloc, device_status);

    TmaMaps maps_x, maps_h;
    if (!make_maps(&maps_x, B.xp16, pl.R_alloc, D.d) || !make_maps(&maps_h, B.h16, pl.R_alloc, D.F))
        return cudaErrorNotSupported;

    for (int mode = 0; mode < 2; ++mode) {
        TcParams p;
        p.D = D; p.L = mode == 0 ? Lgu : Ld; p.P = P; p.mode = mode;
        p.n_cap = pl.n_cap;
        p.n_row_tiles = mode == 0 ? D.F / 64 : D.d / 128;
        p.n_split = mode == 0 ? 1 : pl.n_split;
        p.groups_per_split = mode == 0 ? p.L.n_groups : pl.groups_per_split;
        p.units = B.units; p.n_units = B.n_units; p.next_item = B.n_units + 1 + mode;
        p.hbuf = B.h16; p.obuf = B.o32; p.row_scale = B.slot_f; p.R_alloc = pl.R_alloc; p.status = device_status;
        const int b_bytes = NSB * pl.n_cap * D.g * 2;
        const int w_slot = 2 * p.L.block_bytes;
        const int bar_bytes = 512;
        const int budget = 224 * 1024;
        int nsw = (budget - b_bytes - bar_bytes - 1024) / w_slot;
        if (nsw > MAX_NSW) nsw = MAX_NSW;
        if (nsw < 2) return cudaErrorInvalidConfiguration;
        p.nsw = nsw;
        p.smem_w_off = b_bytes;
        p.smem_bar_off = (b_bytes + nsw * w_slot + 127) & ~127;
        const int smem_bytes = p.smem_bar_off + bar_bytes + 1024;   // + slack for the 1024-byte alignment
        mark(mode == 0 ? 1 : 2);
        // width lists of at most four segments that have a specialised kernel (nibble j = width of segment j)
        int wpack = 0;
        // (every width step stored as one segment; the tied-scale layout has compile-time segment offsets)
        if (p.L.n_seg <= 4 && p.L.n_seg == p.L.n_widths)
            for (int j = 0; j < p.L.n_seg; ++j) wpack |= p.L.seg_w[j] << (4 * j);
        auto launch = [&](auto kc) -> cudaError_t {
            constexpr auto kern = decltype(kc)::value;
            cudaError_t err = ensure_dynamic_smem<kern>(smem_bytes);
            if (err != cudaSuccess) return err;
            launch_chained(kern, dim3(sms), dim3(TC_THREADS), smem_bytes, st, p, mode == 0 ? maps_x : maps_h);
            return cudaSuccess;
        };
#define TC_KERNEL(GS_, WP_) std::integral_constant<decltype(&ffn_tc_kernel<GS_, WP_>), &ffn_tc_kernel<GS_, WP_>>{}
        cudaError_t e;
        if (D.g == 128 && wpack == 0x4112) e = launch(TC_KERNEL(128, 0x4112));        // {2,3,4,8}
        else if (D.g == 128 && wpack == 0x422) e = launch(TC_KERNEL(128, 0x422));     // {2,4,8}
        else if (D.g == 128) e = launch(TC_KERNEL(128, 0));
        else e = launch(TC_KERNEL(64, 0));
#undef TC_KERNEL
        if (e != cudaSuccess) return e;
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}
