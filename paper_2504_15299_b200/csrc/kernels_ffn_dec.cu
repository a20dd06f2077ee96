// Memory-bound grouped dequant kernel for decode-sized expert loads (tcgen05 + TMEM).
//
// Same tile geometry as the grouped dequant-GEMM (128 weight rows on the MMA's M side = TMEM lanes,
// tokens on N, one K-group of g input columns per pipeline stage, thread = weight row), but built
// around the fact that a decode call is bound by HBM bytes and by the two half-rate pipes of the SM
// (integer/logic and packed-fp16 arithmetic) that turn packed codes into MMA operands, not by the
// tensor cores.  So the work per packed code is cut to the minimum, one AND and one packed FMA:
//
//   * The reconstruction rule of Section 3.3.1 is additive over the segments of the nested code,
//         W_hat_b = [lo + s1 v_0] + sum_{1 <= j <= k(b)} M_j (v_j - (2^{w_j} - 1)/2),
//     (v_j = value of segment j, w_j its width, M_j = s1 / 2^(bits[j]-bits[0]); the sum of the
//     constants telescopes to the -s1/2 + s_b/2 of the closed form).  Each bracket is ONE tile:
//     tile_j = code pattern * multiplier + constant, a single packed-fp16 FMA per code pair whose
//     result goes straight to TMEM, with no running sum in registers.
//   * The tokens of a unit are sorted by width, widest first, so the tokens that need segment j are
//     the first n_j rows of the activation tile.  tile_j is multiplied with those rows only
//     (N_j = n_j rounded up to 16) into its own accumulator D_j; the epilogue adds, for every token,
//     the D_j of the segments its width includes.  The extra tensor work (a wide token meets up to
//     K tiles) is free here: the tensor pipe is mostly idle in decode.
//   * Every segment plane is read from HBM once per (unit, row tile) whatever the mix of widths
//     (the plane reuse of Section 3.4), through a deep ring of bulk async copies.
//
// A code pair is isolated by AND inside the fp16 subnormal range, where the bit pattern v << p is the
// value v * 2^(p-24), so the FMA needs no int-to-float conversion.  All tiles carry a common factor
// 2^-S (S per matrix, from the largest scale seen at pack time) so the multipliers stay in fp16
// range; the epilogue multiplies by 2^S.
//
// CTA = 384 threads, 2 CTAs per SM: warps 0-3 and 4-7 are two dequant warpgroups; warpgroup w takes
// the segments w, w+2, ... of every K-group and owns two 32-column operand slots in TMEM that
// alternate; warp 8 streams packed blocks (cp.async.bulk), warp 9 streams activation tiles (TMA,
// 128B swizzle), warps 10 and 11 issue the MMAs of warpgroup 0 and 1.  TMEM per CTA: 128 accumulator columns (K segments x n_cap tokens) + 4 x 32 operand columns.
// Every wait is bounded; on expiry the CTA raises D2MOE_DEV_TIMEOUT, stops waiting, drains, exits.
#include "d2moe_common.cuh"
#include "kernels_ffn_tc.cuh"
#include "tc_common.cuh"

namespace {

constexpr int DEC_THREADS = 384;
constexpr int DEC_WARP_WPROD = 8, DEC_WARP_BPROD = 9, DEC_WARP_MMA = 10;   // MMA issuers: warps 10 and 11
constexpr int DEC_TMEM_COLS = 256;
constexpr int DEC_D_COLS = 128;
constexpr int DEC_NSB = 4;             // activation ring depth
constexpr int DEC_MAX_NSW = 8;         // weight ring depth (upper bound)
constexpr int DEC_EPI_STRIDE = 17;

struct DecParams {
    MoeDims D;
    PackLayout L;
    ExpertPtrs P;
    int mode;                 // 0: gate/up + SwiGLU -> hbuf;  1: down -> obuf
    int n_cap, n_row_tiles, n_split, groups_per_split, nsw;
    const TcUnit* units;
    const int* n_units;
    __half* hbuf;             // [R, F]
    float* obuf;              // [n_split][R, d]
    long long R_alloc;
    int32_t* status;
    int smem_w_off, smem_epi_off, smem_bar_off;
    int dbg;                  // debug builds only: bit 0 skips the MMAs, bit 1 skips the dequant math
};

struct DecItem { int unit, tile, split, g0, g1; };

#ifdef D2MOE_WAIT_STATS
// Debug build only: cycles spent per wait category, summed over all CTAs (read back by
// d2moe_debug_wait_stats).  0 wprod.w_empty 1 bprod.b_empty 2 mma.d_empty 3 mma.b_full 4 mma.a_full
// 5 mma.total 6 deq.w_full 7 deq.a_empty 8 deq.wait_st 9 deq.d_full 10 deq.total 11 deq.epilogue
__device__ unsigned long long g_wait_stats[16];
#define STAT_T0() const long long _t0 = clock64()
#define STAT_ADD(slot) stat[slot] += clock64() - _t0
#define STAT_DECL() long long stat[16] = {0}
#define STAT_FLUSH(cond) do { if (cond) { for (int _i = 0; _i < 16; ++_i) if (stat[_i]) atomicAdd(&g_wait_stats[_i], (unsigned long long)stat[_i]); } } while (0)
#else
#define STAT_T0()
#define STAT_ADD(slot)
#define STAT_DECL()
#define STAT_FLUSH(cond)
#endif

__device__ __forceinline__ DecItem dec_item(const DecParams& p, int item) {
    DecItem it;
    const int per_unit = p.n_row_tiles * p.n_split;
    it.unit = item / per_unit;
    const int rem = item - it.unit * per_unit;
    it.tile = rem / p.n_split;
    it.split = rem - it.tile * p.n_split;
    it.g0 = it.split * p.groups_per_split;
    it.g1 = min(p.L.n_groups, it.g0 + p.groups_per_split);
    return it;
}

// 64 consecutive codes (elements 64h .. 64h+63 of the group) of one segment of one row ->
// 32 half2 registers tile[i] = code pair * multiplier + addend, written to TMEM columns
// [taddr, taddr + 32).   m0: multiplier of a code at bit position 0; position p uses m0 * 2^-p.
template <int SW>
__device__ __forceinline__ void make_multipliers(__half2 m0, __half2 (&mult)[8]) {
    mult[0] = m0;
    const __half2 step = __float2half2_rn(1.0f / (float)(1 << SW));
#pragma unroll
    for (int q = 1; q < 8 / SW; ++q) mult[q] = __hmul2(mult[q - 1], step);
}

template <int GS, int SW>
__device__ __forceinline__ void dequant_half_tile(uint32_t seg, int rr, int h, const __half2 (&mult)[8], __half2 addend, uint32_t taddr) {
    constexpr int ROW_BYTES = GS * SW / 8;
    constexpr int CS = ROW_BYTES < 16 ? ROW_BYTES : 16;      // chunk size of the packed layout
    constexpr int HALF_BYTES = 8 * SW;                       // bytes of 64 codes
    constexpr int LD = HALF_BYTES < 16 ? HALF_BYTES : 16;    // bytes per shared load
    constexpr int NLD = HALF_BYTES / LD;
    constexpr int WPL = LD / 4;                              // words per load
    constexpr int PER = 16 / SW;                             // registers per word
    constexpr int NPOS = 8 / SW;                             // distinct bit positions per byte lane
    constexpr uint32_t FIELD = ((1u << SW) - 1u) * 0x00010001u;

    uint32_t w[NLD * WPL];
#pragma unroll
    for (int l = 0; l < NLD; ++l) {
        const int off = h * HALF_BYTES + l * LD;             // byte offset inside the row's bytes
        const int c = off / CS, within = off % CS;           // (h is a loop constant after unrolling)
        const uint32_t addr = seg + (uint32_t)((c * D2MOE_TILE_ROWS + rr) * CS + within);
        if constexpr (WPL == 4) {
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w[l * 4 + 0]), "=r"(w[l * 4 + 1]), "=r"(w[l * 4 + 2]), "=r"(w[l * 4 + 3]) : "r"(addr));
        } else if constexpr (WPL == 2) {
            asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(w[l * 2 + 0]), "=r"(w[l * 2 + 1]) : "r"(addr));
        } else {
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w[l]) : "r"(addr));
        }
    }
    // two batches of 16 registers, each stored to TMEM as soon as it is complete
#pragma unroll
    for (int b = 0; b < 2; ++b) {
        uint32_t v[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int idx = b * 16 + i, q = idx / PER, e = idx % PER;
            const uint32_t src = (e & 1) ? (w[q] >> 8) : w[q];   // pair e of the word: bytes (0,2) or (1,3), bit SW*(e/2)
            v[i] = as_u32(__hfma2(as_h2(src & (FIELD << ((e >> 1) * SW))), mult[e >> 1], addend));
        }
        tc_st16(taddr + b * 16, v);
    }
}

template <int GS>
__device__ __forceinline__ void dequant_half_dispatch(int sw, uint32_t seg, int rr, int h, __half2 m0, __half2 addend, uint32_t taddr) {
    __half2 mult[8];
    switch (sw) {
        case 1: make_multipliers<1>(m0, mult); dequant_half_tile<GS, 1>(seg, rr, h, mult, addend, taddr); break;
        case 2: make_multipliers<2>(m0, mult); dequant_half_tile<GS, 2>(seg, rr, h, mult, addend, taddr); break;
        case 4: make_multipliers<4>(m0, mult); dequant_half_tile<GS, 4>(seg, rr, h, mult, addend, taddr); break;
        default: make_multipliers<8>(m0, mult); dequant_half_tile<GS, 8>(seg, rr, h, mult, addend, taddr); break;
    }
}

// Compile-time description of a width list whose segments are stored exactly (widths 1, 2, 4, 8):
// nibble j of SWPACK is the width of segment j.  SWPACK == 0 selects the run-time path.
template <int SWPACK>
struct SegList {
    __host__ __device__ static constexpr int sw(int j) { return (SWPACK >> (4 * j)) & 15; }
    __host__ __device__ static constexpr int count() { int k = 0; while (k < 8 && sw(k) != 0) ++k; return k; }
    __host__ __device__ static constexpr int bits_upto(int j) { int b = 0; for (int i = 0; i <= j; ++i) b += sw(i); return b; }
    __host__ __device__ static constexpr int seg_off(int gs, int j) { int o = D2MOE_TILE_ROWS * 4; for (int i = 0; i < j; ++i) o += D2MOE_TILE_ROWS * gs * sw(i) / 8; return o; }
};

// One K-group of warpgroup WG with a compile-time width list: its segments j = WG, WG+2 (at most two
// when the list has at most four), both halves, straight-line code.  fac[q], cfac[q]: per-item factors
// so that multiplier(position 0) = s1 * fac and the tile constant = s1 * cfac (segment 0: lo * 2^-S).
template <int GS, int SWPACK, int WG, typename WaitEmpty, typename Publish>
__device__ __forceinline__ void dequant_group_fixed(int dbg, uint32_t wb, int rr, int kmax, float s1, float lo_scaled,
                                                    const float (&fac)[2], const float (&cfac)[2], uint32_t a_slots,
                                                    WaitEmpty&& wait_empty, Publish&& publish) {
    using SL = SegList<SWPACK>;
    constexpr int HALVES = GS / 64;
    __half2 mult[2][8];
    __half2 addend[2];
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        constexpr int dummy = 0; (void)dummy;
        const int j = WG + 2 * q;
        if (j < SL::count()) {
            const __half2 m0 = __float2half2_rn(s1 * fac[q]);
            if (SL::sw(j < 8 ? j : 0) == 1) make_multipliers<1>(m0, mult[q]);
            else if (SL::sw(j < 8 ? j : 0) == 2) make_multipliers<2>(m0, mult[q]);
            else if (SL::sw(j < 8 ? j : 0) == 4) make_multipliers<4>(m0, mult[q]);
            else make_multipliers<8>(m0, mult[q]);
            addend[q] = __float2half2_rn(j == 0 ? lo_scaled : s1 * cfac[q]);
        }
    }
#pragma unroll 1
    for (int h = 0; h < HALVES; ++h) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            constexpr int K = SL::count();
            const int j = WG + 2 * q;
            if (j < K) {
                if (j <= kmax) {
                    wait_empty(q);
                    const uint32_t seg = wb + (uint32_t)SL::seg_off(GS, j < 8 ? j : 0);
                    const uint32_t taddr = a_slots + q * 32;
#ifdef D2MOE_WAIT_STATS
                    if (dbg & 2) { publish(q); continue; }
#endif
                    if (SL::sw(j < 8 ? j : 0) == 1) dequant_half_tile<GS, 1>(seg, rr, h, mult[q], addend[q], taddr);
                    else if (SL::sw(j < 8 ? j : 0) == 2) dequant_half_tile<GS, 2>(seg, rr, h, mult[q], addend[q], taddr);
                    else if (SL::sw(j < 8 ? j : 0) == 4) dequant_half_tile<GS, 4>(seg, rr, h, mult[q], addend[q], taddr);
                    else dequant_half_tile<GS, 8>(seg, rr, h, mult[q], addend[q], taddr);
                    publish(q);
                }
            }
        }
    }
}

template <int GS, int SWPACK>
__global__ void __launch_bounds__(DEC_THREADS, 2)
ffn_dec_kernel(const __grid_constant__ DecParams p, const __grid_constant__ TmaMaps maps) {
    constexpr int HALVES = GS / 64;
    extern __shared__ uint8_t smem_raw[];
    // shared layout from a 1024-byte boundary:
    // [activation ring: DEC_NSB x n_cap*GS*2] [weight ring: nsw x 2 blocks] [epilogue x2] [barriers]
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t b_slot_bytes = (uint32_t)p.n_cap * GS * 2;
    const uint32_t w_slot_bytes = 2u * (uint32_t)p.L.block_bytes;
    const uint32_t bbuf = smem_base;
    const uint32_t wbuf = smem_base + p.smem_w_off;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.smem_bar_off);
    const uint32_t bar0 = smem_u32(bars);
    auto W_FULL = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    auto W_EMPTY = [&](int i) { return bar0 + 8u * (uint32_t)(DEC_MAX_NSW + i); };
    auto B_FULL = [&](int i) { return bar0 + 8u * (uint32_t)(2 * DEC_MAX_NSW + i); };
    auto B_EMPTY = [&](int i) { return bar0 + 8u * (uint32_t)(2 * DEC_MAX_NSW + DEC_NSB + i); };
    auto A_FULL = [&](int wg, int sl) { return bar0 + 8u * (uint32_t)(2 * DEC_MAX_NSW + 2 * DEC_NSB + wg * 2 + sl); };
    auto A_EMPTY = [&](int wg, int sl) { return bar0 + 8u * (uint32_t)(2 * DEC_MAX_NSW + 2 * DEC_NSB + 4 + wg * 2 + sl); };
    const uint32_t D_FULL = bar0 + 8u * (uint32_t)(2 * DEC_MAX_NSW + 2 * DEC_NSB + 8);
    const uint32_t D_EMPTY = D_FULL + 8u;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * DEC_MAX_NSW + 2 * DEC_NSB + 10);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < DEC_MAX_NSW; ++i) { mbar_init(W_FULL(i), 1); mbar_init(W_EMPTY(i), 256); }
        for (int i = 0; i < DEC_NSB; ++i) { mbar_init(B_FULL(i), 1); mbar_init(B_EMPTY(i), 2); }
        for (int wg = 0; wg < 2; ++wg)
            for (int sl = 0; sl < 2; ++sl) { mbar_init(A_FULL(wg, sl), 128); mbar_init(A_EMPTY(wg, sl), 1); }
        mbar_init(D_FULL, 2);
        mbar_init(D_EMPTY, 256);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == DEC_WARP_MMA) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(DEC_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t d_tmem = tmem_base;                        // segment j: columns [j*n_cap, (j+1)*n_cap)
    const uint32_t a_tmem = tmem_base + DEC_D_COLS;           // warpgroup wg, slot sl: + (wg*2 + sl)*32

    const int n_units = *p.n_units;
    const int total_items = n_units * p.n_row_tiles * p.n_split;
    const int nsw = p.nsw;

    if (warp == DEC_WARP_WPROD) {
        if (lane == 0) {
            STAT_DECL();
            uint32_t it = 0;
            for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
                const DecItem ii = dec_item(p, item);
                const TcUnit* u = p.units + ii.unit;
                const int e = u->e, kmax = u->kmax;
                const uint32_t bytes = (uint32_t)p.L.seg_off[kmax + 1];
                const uint8_t *m0, *m1;
                int rt0, rt1;
                if (p.mode == 0) { m0 = p.P.w[3 * e + 0]; m1 = p.P.w[3 * e + 1]; rt0 = rt1 = ii.tile; }
                else { m0 = m1 = p.P.w[3 * e + 2]; rt0 = 2 * ii.tile; rt1 = 2 * ii.tile + 1; }
                for (int G = ii.g0; G < ii.g1; ++G, ++it) {
                    const int s = it % nsw;
                    { STAT_T0(); mbar_wait(W_EMPTY(s), ((it / nsw) & 1) ^ 1, abort_flag, p.status); STAT_ADD(0); }
                    mbar_expect_tx(W_FULL(s), 2 * bytes);
                    const uint32_t dst = wbuf + s * w_slot_bytes;
                    bulk_g2s(dst, m0 + d2moe_block_offset(p.L, rt0, G), bytes, W_FULL(s));
                    bulk_g2s(dst + p.L.block_bytes, m1 + d2moe_block_offset(p.L, rt1, G), bytes, W_FULL(s));
                }
            }
            for (int s = 0; s < nsw && s < (int)it; ++s) {      // drain: all copies issued have landed
                const uint32_t last = it - 1 - (it - 1 - s) % nsw;
                mbar_wait(W_FULL(s), (last / nsw) & 1, abort_flag, p.status, true);
            }
            STAT_FLUSH(true);
        }
    } else if (warp == DEC_WARP_BPROD) {
        if (lane == 0) {
            STAT_DECL();
            uint32_t it = 0;
            for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
                const DecItem ii = dec_item(p, item);
                const TcUnit* u = p.units + ii.unit;
                int mi = 0, box = 16;
                while (box < u->ncols) { box <<= 1; ++mi; }
                const uint32_t bytes = (uint32_t)box * 128u * HALVES;
                for (int G = ii.g0; G < ii.g1; ++G, ++it) {
                    const int s = it % DEC_NSB;
                    { STAT_T0(); mbar_wait(B_EMPTY(s), ((it / DEC_NSB) & 1) ^ 1, abort_flag, p.status); STAT_ADD(1); }
                    mbar_expect_tx(B_FULL(s), bytes);
                    const uint32_t dst = bbuf + s * b_slot_bytes;
#pragma unroll
                    for (int h = 0; h < HALVES; ++h)
                        tma_load_2d(dst + h * (uint32_t)p.n_cap * 128u, &maps.m[mi], G * GS + h * 64, u->row0, B_FULL(s));
                }
            }
            for (int s = 0; s < DEC_NSB && s < (int)it; ++s) {
                const uint32_t last = it - 1 - (it - 1 - s) % DEC_NSB;
                mbar_wait(B_FULL(s), (last / DEC_NSB) & 1, abort_flag, p.status, true);
            }
            STAT_FLUSH(true);
        }
    } else if (warp >= DEC_WARP_MMA) {
        // Two MMA issuers, one per dequant warpgroup: issuer w multiplies the tiles warpgroup w writes
        // (segments w, w+2, ...: accumulators disjoint from the other issuer's) from that warpgroup's two
        // operand slots, which alternate, so a slot is refilled while the other one is being multiplied.
        // One thread issues at most one tcgen05.mma per ~45 cycles whatever its size, so the issue work
        // is split over two warps.  The whole warp runs the loop and one elected lane issues, so that
        // addresses and descriptors stay in the uniform datapath (fewer instructions per MMA, which
        // matters because the issuer competes with the dequant warps for issue slots).
        {
            STAT_DECL();
#ifdef D2MOE_WAIT_STATS
            const long long _tt = clock64();
#endif
            const int w = warp - DEC_WARP_MMA;
            uint32_t it = 0, ic = 0;
            uint32_t use0 = 0, use1 = 0;                     // uses of slot 0 / 1 of warpgroup w
            const uint32_t n_cap_bytes = (uint32_t)p.n_cap * 128u;
            const uint32_t a_slot0 = a_tmem + (w * 2) * 32, a_slot1 = a_slot0 + 32;
            for (int item = blockIdx.x; item < total_items; item += gridDim.x, ++ic) {
                const DecItem ii = dec_item(p, item);
                const TcUnit* u = p.units + ii.unit;
                const int kmax = u->kmax;
                const int n_mine = kmax >= w ? (kmax - w) / 2 + 1 : 0;       // segments w, w+2, ...
                uint32_t idesc[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) idesc[q] = instr_desc_f16(u->cnt[(2 * q + w) & 7]);
                { STAT_T0(); mbar_wait(D_EMPTY, (ic & 1) ^ 1, abort_flag, p.status); STAT_ADD(2); }
                tc_fence_after();
                for (int G = ii.g0; G < ii.g1; ++G, ++it) {
                    const int s = it % DEC_NSB;
                    { STAT_T0(); mbar_wait(B_FULL(s), (it / DEC_NSB) & 1, abort_flag, p.status); STAT_ADD(3); }
                    const uint64_t bdesc = smem_desc_sw128(bbuf + s * b_slot_bytes);
                    const uint32_t first = (G != ii.g0) ? 1u : 0u;
#pragma unroll 1
                    for (int qp = 0; qp < 2; ++qp) {                  // pairs of my segments: slots 0 and 1
#pragma unroll 1
                        for (int h = 0; h < HALVES; ++h) {
#pragma unroll
                            for (int sl = 0; sl < 2; ++sl) {
                                const int q = 2 * qp + sl;
                                if (q < n_mine) {
                                    const uint32_t idq = q == 0 ? idesc[0] : q == 1 ? idesc[1] : q == 2 ? idesc[2] : idesc[3];
                                    const uint32_t d_addr = d_tmem + (2 * q + w) * p.n_cap;
                                    const uint32_t a_addr = sl ? a_slot1 : a_slot0;
                                    const uint32_t use = sl ? use1 : use0;
                                    { STAT_T0(); mbar_wait(A_FULL(w, sl), use & 1, abort_flag, p.status); STAT_ADD(4); }
                                    tc_fence_after();
                                    const uint64_t bh = bdesc + (uint64_t)((h * n_cap_bytes) >> 4);
                                    {
                                        STAT_T0();
                                        if (elect_one()) {
#ifdef D2MOE_WAIT_STATS
                                            if (!(p.dbg & 1))
#endif
                                            {
                                                tc_mma_ts(d_addr, a_addr + 0, bh + 0, idq, h == 0 ? first : 1u);
                                                tc_mma_ts(d_addr, a_addr + 8, bh + 2, idq, 1u);
                                                tc_mma_ts(d_addr, a_addr + 16, bh + 4, idq, 1u);
                                                tc_mma_ts(d_addr, a_addr + 24, bh + 6, idq, 1u);
                                            }
                                            tc_commit(A_EMPTY(w, sl));
                                        }
                                        __syncwarp();
                                        STAT_ADD(12);
#ifdef D2MOE_WAIT_STATS
                                        stat[13] += 1;
#endif
                                    }
                                    if (sl) ++use1; else ++use0;
                                }
                            }
                        }
                    }
                    if (elect_one()) tc_commit(B_EMPTY(s));
                    __syncwarp();
                }
                if (elect_one()) tc_commit(D_FULL);
                __syncwarp();
            }
            if (ic > 0) mbar_wait(D_FULL, (ic - 1) & 1, abort_flag, p.status, true);
#ifdef D2MOE_WAIT_STATS
            stat[5] = clock64() - _tt;
#endif
            STAT_FLUSH(w == 0 && lane == 0);
        }
    } else {
        // -------- two dequant warpgroups (warpgroup w: segments w, w+2, ... of every K-group) + epilogue --------
        const int wg = warp >> 2;
        const int r = threadIdx.x & 127;           // row of the tile = TMEM lane
        const int blk = r >> 6, rr = r & 63;
        const uint32_t lane_addr = ((uint32_t)((warp & 3) * 32)) << 16;
        float* epi = reinterpret_cast<float*>(smem + p.smem_epi_off) + wg * (64 * DEC_EPI_STRIDE);
        uint32_t it = 0, ic = 0, use0 = 0, use1 = 0;       // use counts of this warpgroup's operand slots
        STAT_DECL();
#ifdef D2MOE_WAIT_STATS
        const long long _tt = clock64();
#endif
        for (int item = blockIdx.x; item < total_items; item += gridDim.x, ++ic) {
            const DecItem ii = dec_item(p, item);
            const TcUnit* u = p.units + ii.unit;
            const int e = u->e, kmax = u->kmax;
            const uint8_t* mat = p.mode == 0 ? p.P.w[3 * e + blk] : p.P.w[3 * e + 2];
            const int S = matrix_exponent(mat);
            const float two_mS = exp2f((float)-S);

            // per-item factors of my segments (compile-time width list only)
            float fac[2] = {0.0f, 0.0f}, cfac[2] = {0.0f, 0.0f};
            if constexpr (SWPACK != 0) {
                using SL = SegList<SWPACK>;
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const int j = wg + 2 * q;
                    if (j < SL::count()) {
                        const int delta = (wg == 0 ? SL::bits_upto(2 * q < 8 ? 2 * q : 0) : SL::bits_upto(2 * q + 1 < 8 ? 2 * q + 1 : 0)) - SL::sw(0);
                        const int wj = wg == 0 ? SL::sw(2 * q < 8 ? 2 * q : 0) : SL::sw(2 * q + 1 < 8 ? 2 * q + 1 : 0);
                        const float Mfac = exp2f((float)(-delta - S));                 // M_j 2^-S = s1 * Mfac
                        fac[q] = Mfac * 16777216.0f;
                        cfac[q] = -0.5f * (float)((1 << wj) - 1) * Mfac;
                    }
                }
            }

            for (int G = ii.g0; G < ii.g1; ++G, ++it) {
                const int s = it % nsw;
                { STAT_T0(); mbar_wait(W_FULL(s), (it / nsw) & 1, abort_flag, p.status); STAT_ADD(6); }
                const uint32_t wb = wbuf + s * w_slot_bytes + blk * p.L.block_bytes;
                uint32_t meta;
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(meta) : "r"(wb + 4u * rr));
                const __half2 mh = as_h2(meta);
                const float s1 = __low2float(mh) * two_mS, lo = __high2float(mh) * two_mS;
                if constexpr (SWPACK != 0) {
                    auto wait_empty = [&](int sl) {
                        const uint32_t use = sl ? use1 : use0;
                        STAT_T0(); mbar_wait(A_EMPTY(wg, sl), (use & 1) ^ 1, abort_flag, p.status); STAT_ADD(7);
                        tc_fence_after();
                    };
                    auto publish = [&](int sl) {
                        tc_wait_st();
                        tc_fence_before();
                        mbar_arrive(A_FULL(wg, sl));
                        if (sl) ++use1; else ++use0;
                    };
                    const float s1raw = __low2float(mh);
                    if (wg == 0) dequant_group_fixed<GS, SWPACK, 0>(p.dbg, wb, rr, kmax, s1raw, lo, fac, cfac, a_tmem + lane_addr, wait_empty, publish);
                    else dequant_group_fixed<GS, SWPACK, 1>(p.dbg, wb, rr, kmax, s1raw, lo, fac, cfac, a_tmem + 64 + lane_addr, wait_empty, publish);
                } else {
                // my segments j = wg + 2q, in pairs: q = 2qp + sl fills operand slot sl
                    const int n_mine = kmax >= wg ? (kmax - wg) / 2 + 1 : 0;
#pragma unroll 1
                    for (int qp = 0; 2 * qp < n_mine; ++qp) {
                        __half2 m0[2], addend[2];
                        uint32_t seg[2];
                        int sw[2];
#pragma unroll
                        for (int sl = 0; sl < 2; ++sl) {
                            const int j = min(wg + 2 * (2 * qp + sl), kmax);
                            sw[sl] = p.L.seg_sw[j];
                            // M_j 2^-S, the position-0 multiplier M_j 2^(24-S), and the tile's constant
                            const float Mj = s1 * exp2f((float)(-(p.D.bits[j] - p.D.bits[0])));
                            m0[sl] = h2dup(Mj * 16777216.0f);
                            addend[sl] = h2dup(j == 0 ? lo : -0.5f * (float)((1 << p.L.seg_w[j]) - 1) * Mj);
                            seg[sl] = wb + (uint32_t)p.L.seg_off[j];
                        }
#pragma unroll
                        for (int h = 0; h < HALVES; ++h) {
#pragma unroll
                            for (int sl = 0; sl < 2; ++sl) {
                                if (2 * qp + sl < n_mine) {
                                    const uint32_t use = sl ? use1 : use0;
                                    { STAT_T0(); mbar_wait(A_EMPTY(wg, sl), (use & 1) ^ 1, abort_flag, p.status); STAT_ADD(7); }
                                    tc_fence_after();
                                    {
                                        STAT_T0();
                                        dequant_half_dispatch<GS>(sw[sl], seg[sl], rr, h, m0[sl], addend[sl],
                                                                  a_tmem + (wg * 2 + sl) * 32 + lane_addr);
                                        STAT_ADD(14);
#ifdef D2MOE_WAIT_STATS
                                        stat[15] += 1;
#endif
                                    }
                                    { STAT_T0(); tc_wait_st(); STAT_ADD(8); }
                                    tc_fence_before();
                                    mbar_arrive(A_FULL(wg, sl));
                                    if (sl) ++use1; else ++use0;
                                }
                            }
                        }
                    }
                }
                mbar_arrive(W_EMPTY(s));
            }

            // ---- epilogue: out[row, token] = 2^S * sum over the segments the token's width includes ----
            { STAT_T0(); mbar_wait(D_FULL, ic & 1, abort_flag, p.status); STAT_ADD(9); }
            tc_fence_after();
#ifdef D2MOE_WAIT_STATS
            const long long _te = clock64();
#endif
            const float two_S = exp2f((float)S);
            const int ncols = u->ncols;
            int nreal[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) nreal[j] = j <= kmax ? u->real[j] : 0;
            for (int c0 = wg * 16; c0 < ncols; c0 += 32) {        // the two warpgroups take alternate chunks
                const int n_tok = min(16, nreal[0] - c0);          // real tokens in this chunk
                if (n_tok <= 0) continue;
                float acc[16];
#pragma unroll
                for (int q = 0; q < 16; ++q) acc[q] = 0.0f;
                for (int j = 0; j <= kmax; ++j) {
                    const int nj = nreal[j] - c0;                  // tokens of this chunk that include segment j
                    if (nj <= 0) break;                            // widths descend along the rows
                    uint32_t v[16];
                    tc_ld16(d_tmem + lane_addr + j * p.n_cap + c0, v);
                    tc_wait_ld();
#pragma unroll
                    for (int q = 0; q < 16; ++q)
                        if (q < nj) acc[q] += __uint_as_float(v[q]);
                }
                const long long grow = u->row0 + c0;
                if (p.mode == 0) {
                    if (blk == 1) {
#pragma unroll
                        for (int q = 0; q < 16; ++q) epi[rr * DEC_EPI_STRIDE + q] = acc[q] * two_S;
                    }
                    asm volatile("bar.sync %0, 128;" ::"r"(1 + wg) : "memory");
                    if (blk == 0) {
                        __half* dst = p.hbuf + grow * p.D.F + (long long)ii.tile * 64 + rr;
#pragma unroll
                        for (int q = 0; q < 16; ++q) {
                            if (q < n_tok) {
                                const float g = acc[q] * two_S;
                                const float up = epi[rr * DEC_EPI_STRIDE + q];
                                dst[(long long)q * p.D.F] = __float2half_rn(g / (1.0f + __expf(-g)) * up);
                            }
                        }
                    }
                    asm volatile("bar.sync %0, 128;" ::"r"(1 + wg) : "memory");
                } else {
                    float* dst = p.obuf + (long long)ii.split * p.R_alloc * p.D.d + grow * p.D.d + (long long)ii.tile * 128 + r;
#pragma unroll
                    for (int q = 0; q < 16; ++q)
                        if (q < n_tok) dst[(long long)q * p.D.d] = acc[q] * two_S;
                }
            }
            tc_fence_before();
            mbar_arrive(D_EMPTY);
#ifdef D2MOE_WAIT_STATS
            stat[11] += clock64() - _te;
#endif
        }
#ifdef D2MOE_WAIT_STATS
        stat[10] = clock64() - _tt;
#endif
        STAT_FLUSH((threadIdx.x & 127) == 0);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == DEC_WARP_MMA) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(DEC_TMEM_COLS) : "memory");
    }
}

// One block.  Lays every expert's tokens out widest width first, pads each expert to a multiple of
// 16 rows, cuts it into units of at most n_cap rows and records, per unit and segment j, how many of
// its rows carry a width that includes segment j (they are the first rows of the unit).
__global__ void __launch_bounds__(256)
dec_prep_kernel(MoeDims D, RouteBufs R, int n_cap, TcUnit* units, int* n_units, int32_t* pad_off,
                int32_t* row_map, int32_t* src_token, int max_units) {
    __shared__ int s_total_rows;
    const int n_exp = D.E + D.n_shared;
    if (threadIdx.x < 32) {                       // padded expert offsets (one warp scans)
        const int lane = threadIdx.x;
        int carry = 0;
        for (int base = 0; base < n_exp; base += 32) {
            const int e = base + lane;
            int n = 0;
            if (e < D.E) n = R.group_off[(e + 1) * D.K] - R.group_off[e * D.K];
            else if (e < n_exp) n = D.T;
            const int v = (n + 15) & ~15;
            int incl = v;
            for (int off = 1; off < 32; off <<= 1) {
                const int o = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += o;
            }
            if (e < n_exp) pad_off[e] = carry + incl - v;
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) { pad_off[n_exp] = carry; s_total_rows = carry; }
    }
    __syncthreads();
    const int total_rows = s_total_rows;
    for (int i = threadIdx.x; i < total_rows; i += blockDim.x) src_token[i] = -1;
    __syncthreads();
    for (int a = threadIdx.x; a < D.A; a += blockDim.x) {
        const int pos = R.inv_perm[a];
        const int e = R.topk_idx[a], kk = R.bit_idx[a];
        if (e < 0 || e >= D.E || kk < 0 || kk >= D.K || pos < 0 || pos >= D.A) { row_map[a] = 0; continue; }
        // rows of wider pieces come first: offset = assignments of this expert with a larger width index
        const int wider = R.group_off[(e + 1) * D.K] - R.group_off[e * D.K + kk + 1];
        const int row = pad_off[e] + wider + (pos - R.group_off[e * D.K + kk]);
        row_map[a] = row;
        if (row >= 0 && row < total_rows) src_token[row] = a / D.k;
    }
    for (int i = threadIdx.x; i < D.n_shared * D.T; i += blockDim.x) {
        const int s = i / D.T, t = i - s * D.T;
        const int row = pad_off[D.E + s] + t;
        row_map[D.A + i] = row;
        src_token[row] = t;
    }
    if (threadIdx.x == 0) {
        int nu = 0;
        for (int e = 0; e < n_exp; ++e) {
            const int p0 = pad_off[e], p1 = pad_off[e + 1];
            for (int start = p0; start < p1 && nu < max_units; start += n_cap) {
                const int len = min(p1 - start, n_cap);
                TcUnit u;
                u.e = e; u.row0 = start; u.ncols = len; u.kmax = 0;
                for (int j = 0; j < 8; ++j) {
                    u.col0[j] = j * n_cap; u.cnt[j] = 0; u.real[j] = 0;
                    if (j >= D.K) continue;
                    // C_j = rows of this expert whose width index is >= j (they are rows [0, C_j))
                    const int Cj = e < D.E ? R.group_off[(e + 1) * D.K] - R.group_off[e * D.K + j] : D.T;
                    const int nj = max(0, min(len, Cj - (start - p0)));
                    u.real[j] = nj;
                    u.cnt[j] = (nj + 15) & ~15;
                    if (nj > 0) u.kmax = j;
                }
                if (u.real[0] > 0) units[nu++] = u;
            }
        }
        *n_units = nu;
    }
}

// xp16[row, :] = fp16(x[src_token[row], :]) for real rows (padding rows are never consumed).
__global__ void __launch_bounds__(256)
dec_gather_kernel(int d, const __nv_bfloat16* __restrict__ x, const int32_t* __restrict__ src_token,
                  const int32_t* __restrict__ pad_off, int n_off, __half* __restrict__ xp16) {
    const int total_rows = pad_off[n_off];
    for (int row = blockIdx.x; row < total_rows; row += gridDim.x) {
        const int t = src_token[row];
        if (t < 0) continue;
        const __nv_bfloat162* src = reinterpret_cast<const __nv_bfloat162*>(x + (size_t)t * d);
        __half2* dst = reinterpret_cast<__half2*>(xp16 + (size_t)row * d);
        for (int i = threadIdx.x; i < d / 2; i += blockDim.x) {
            const float2 f = __bfloat1622float2(src[i]);
            dst[i] = __floats2half2_rn(f.x, f.y);
        }
    }
}

}  // namespace

static int g_host_dbg_mode = 0;
#ifdef D2MOE_WAIT_STATS
extern "C" int d2moe_debug_set_mode(int mode) { g_host_dbg_mode = mode; return 0; }
extern "C" int d2moe_debug_wait_stats(unsigned long long* host16, int reset) {
    cudaDeviceSynchronize();
    if (cudaMemcpyFromSymbol(host16, g_wait_stats, sizeof(unsigned long long) * 16) != cudaSuccess) return 1;
    if (reset) { unsigned long long z[16] = {0}; cudaMemcpyToSymbol(g_wait_stats, z, sizeof(z)); }
    return 0;
}
#endif

cudaError_t launch_ffn_decode(const d2moe_config* c, const MoeDims& D, const PackLayout& Lgu, const PackLayout& Ld,
                              const ExpertPtrs& P, const __nv_bfloat16* x, const RouteBufs& R, const TcPlan& pl,
                              const TcBuffers& B, int32_t* device_status, cudaStream_t st, void* const* ev) {
    auto mark = [&](int i) { if (ev) cudaEventRecord((cudaEvent_t)ev[i], st); };
    const int n_exp = D.E + D.n_shared;
    dec_prep_kernel<<<1, 256, 0, st>>>(D, R, pl.n_cap, B.units, B.n_units, B.pad_off, B.row_map, B.src_token, pl.max_units);
    dec_gather_kernel<<<296, 256, 0, st>>>(D.d, x, B.src_token, B.pad_off, n_exp, B.xp16);

    TmaMaps maps_x, maps_h;
    if (!make_maps(&maps_x, B.xp16, pl.R_alloc, D.d) || !make_maps(&maps_h, B.h16, pl.R_alloc, D.F))
        return cudaErrorNotSupported;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);

    for (int mode = 0; mode < 2; ++mode) {
        DecParams p;
        p.D = D; p.L = mode == 0 ? Lgu : Ld; p.P = P; p.mode = mode;
        p.n_cap = pl.n_cap;
        p.n_row_tiles = mode == 0 ? D.F / 64 : D.d / 128;
        p.n_split = mode == 0 ? 1 : pl.n_split;
        p.groups_per_split = mode == 0 ? p.L.n_groups : pl.groups_per_split;
        p.units = B.units; p.n_units = B.n_units;
        p.hbuf = B.h16; p.obuf = B.o32; p.R_alloc = pl.R_alloc; p.status = device_status;
        p.dbg = g_host_dbg_mode;
        const int b_bytes = DEC_NSB * pl.n_cap * D.g * 2;
        const int w_slot = 2 * p.L.block_bytes;
        const int epi_bytes = 2 * 64 * DEC_EPI_STRIDE * 4;
        const int bar_bytes = 512;
        const int budget = 112 * 1024;
        int nsw = (budget - b_bytes - epi_bytes - bar_bytes - 1024) / w_slot;
        if (nsw > DEC_MAX_NSW) nsw = DEC_MAX_NSW;
        if (nsw < 2) return cudaErrorInvalidConfiguration;
        p.nsw = nsw;
        p.smem_w_off = b_bytes;
        p.smem_epi_off = (b_bytes + nsw * w_slot + 127) & ~127;
        p.smem_bar_off = (p.smem_epi_off + epi_bytes + 127) & ~127;
        const int smem_bytes = p.smem_bar_off + bar_bytes + 1024;
        mark(mode == 0 ? 1 : 2);
        // width lists whose segments are stored exactly get a kernel specialised on the list
        int swpack = 0;
        bool exact = p.L.n_seg <= 4;
        for (int j = 0; j < p.L.n_seg && exact; ++j) {
            exact = p.L.seg_w[j] == p.L.seg_sw[j];
            swpack |= p.L.seg_sw[j] << (4 * j);
        }
        if (!exact) swpack = 0;
        auto launch = [&](auto kern) -> cudaError_t {
            cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
            if (err != cudaSuccess) return err;
            kern<<<2 * sms, DEC_THREADS, smem_bytes, st>>>(p, mode == 0 ? maps_x : maps_h);
            return cudaSuccess;
        };
        cudaError_t e;
        if (D.g == 128 && swpack == 0x4112) e = launch(ffn_dec_kernel<128, 0x4112>);
        else if (D.g == 128 && swpack == 0x422) e = launch(ffn_dec_kernel<128, 0x422>);
        else if (D.g == 64 && swpack == 0x422) e = launch(ffn_dec_kernel<64, 0x422>);
        else if (D.g == 128) e = launch(ffn_dec_kernel<128, 0>);
        else e = launch(ffn_dec_kernel<64, 0>);
        if (e != cudaSuccess) return e;
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}
