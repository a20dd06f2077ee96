// Memory-bound expert kernel for decode-sized loads: 8-bit tensor-core products on the packed codes
// themselves, scales applied to the accumulators (tcgen05 kind::i8 + TMEM).
//
// The reconstruction rule of Section 3.3.1 in closed form, for a token routed at width b (index kk),
//     W_hat_b[r, k] = lo + s1 * ( Q_b[r, k] * 2^-(top - b1) + 2^-(b - b1 + 1) - 1/2 ),
// where Q_b is the nested top-width code with the bits below width b cleared (the sum of the
// segments 0..kk, each at its position inside the top-width code), (s1, lo) belong to (row, group)
// and b1 / top are the narrowest / widest width.  With the activations of a token written as
// x[k] = sigma * xq[k] (xq a 15-bit integer, sigma per token), one output element is
//     y[r] = sigma * sum_G { s1' * ( sum_{k in G} Q_b[r, k] xq[k]  +  kappa_b X_G )  +  lo * X_G },
//     s1' = s1 * 2^-(top - b1),  kappa_b = 2^(top - b - 1) - 2^(top - b1 - 1),  X_G = sum_{k in G} xq[k].
// The inner sum is an exact integer contraction: the tensor cores run it on unsigned 8-bit codes
// and signed 8-bit activation halves (xq = 128 hi + lo8), so the CUDA cores never expand a code to
// a floating-point weight.  What is left for them per packed word is one shift and one AND per four
// codes (the packed layout keeps the four codes of an operand cell in the four bytes of a word), and
// per (row, group, token) four instructions that fold the accumulator into the running output
// (128 hi + lo8, int -> float, acc += s1' D, acc += (s1' kappa_b + lo) X_G: the bracket once per block
// of four slots, which share a width).
//
//   * The tokens of a unit are laid out by width, widest first, each width class padded to 8 slots:
//     the slots that include segment j are the first npad[j] of the unit, and the product of
//     segment j runs over exactly those (N = 2 npad[j]: a high and a low activation row per slot).
//     All segments of a group accumulate into ONE accumulator, each at its position in the code.
//   * Every segment plane is read from HBM once per (unit, row tile) whatever the mix of widths
//     (the plane reuse of Section 3.4), through a ring of bulk async copies; a unit whose widest
//     token is narrower than the top width reads only the prefix it needs.
//   * The accumulator is double buffered per group: while the products of group G+1 run, the
//     fold warps add group G to their fp32 registers.
//
// Two instantiations per width list, 2 CTAs per SM either way; thread = weight row = TMEM lane in every warpgroup.
// Warps 0-3 unpack: per group they fill operand slot 0 (segments 0 and 2 of the group, two 32-column tiles in TMEM)
// and hand it to the issuer, then slot 1 (segments 1 and 3).  Then the fold warps: two warpgroups (CTA = 448
// threads, 72 registers), each taking half of the unit's token blocks, when the units are full; one warpgroup
// (CTA = 320 threads, 96 registers) that takes all blocks when a unit holds few tokens (fewer waiting warps: 4-5 %
// faster up to about 12 tokens per expert, slower beyond).  The fold warps also run the output phase of a work item.
// Then one warp that streams packed blocks (cp.async.bulk), activation tiles (TMA, 128B swizzle) and the per-group
// activation sums, and one that issues the MMAs.  TMEM per CTA: 2 x 64 accumulator columns + 4 x 32 operand columns.
//
// Work distribution: a work item is one unit x one tile of 128 weight rows x a range of groups.  The
// producer thread takes item numbers from a global counter (which starts at the grid size: item i < grid
// belongs to CTA i) and publishes them to the other warps through a small queue in shared memory; the
// units are ordered by decreasing work, so the cheap items are drawn last.
//
// Every wait is bounded (barriers only, no bar.sync inside the roles); on expiry the CTA raises
// D2MOE_DEV_TIMEOUT, stops waiting, drains its copies, frees its TMEM and exits.
#include "d2moe_common.cuh"
#include "kernels_ffn_tc.cuh"
#include "tc_common.cuh"
#include "group_block.cuh"

#include <type_traits>

namespace {

// Warps: 0-3 unpack, then NF fold warpgroups (1 or 2), the producer warp, the issuer warp.  Two fold warpgroups
// (each half of the unit's token blocks, 72 registers) win when the units are full; one (all blocks, 96 registers,
// fewer waiting warps) when a unit holds few tokens.
__host__ __device__ constexpr int i8_threads(int nf) { return 32 * (4 + 4 * nf + 2); }
constexpr int I8_TMEM_COLS = 256;
constexpr int I8_D_COLS = 64;                 // one accumulator buffer: 32 slots x (high, low)
constexpr int I8_SLOTS = 32;                  // token slots per unit
constexpr int I8_NSB = 4;                     // activation ring depth
constexpr int I8_MAX_NSW = 8;                 // weight ring depth (upper bound)
constexpr int I8_B_TILE = 2 * I8_SLOTS * 128; // 64 rows x 128 bytes (128 input columns)
constexpr int I8_XK_BYTES = I8_SLOTS * 8;     // (X, kappa) per slot, one group
constexpr int I8_B_STAGE = I8_B_TILE + 2 * I8_XK_BYTES;
constexpr int I8_NSQ = 4;                     // entries of the work queue between the producer and the other warps
// barriers: weight ring (full, empty), activation ring (full, empty), 4 + 4 hand-offs, 2 + 2 accumulators,
// work queue (full, empty)
constexpr int I8_N_BARS = 2 * I8_MAX_NSW + 2 * I8_NSB + 12 + 2 * I8_NSQ;
constexpr float I8_XMAX = 16191.0f;           // |xq| <= 126 * 128 + 63

struct I8Params {
    MoeDims D;
    PackLayout L;
    ExpertPtrs P;
    int mode;                 // 0: gate/up + SwiGLU -> hbuf;  1: down -> obuf
    int n_row_tiles, n_split, groups_per_split, nsw;
    const I8Unit* units;
    const int* n_units;
    int* next_item;           // work counter of this launch: starts at the grid size (item i < grid goes to CTA i)
    const float* xk;          // [n_groups][R_alloc][2]
    const float* sigma;       // [R_alloc]
    float* hbuf;              // [R_alloc, F]
    float* obuf;              // [n_split][R_alloc, d]
    long long R_alloc;
    int32_t* status;
    int smem_w_off, smem_rec_off, smem_bar_off;
};

struct I8Item { int unit, tile, split, g0, g1; };
struct I8SegMap { int n_seg; int seg_kk[8]; };   // stored segment -> width index of the step it belongs to


__device__ __forceinline__ I8Item i8_item(const I8Params& p, int item) {
    I8Item it;
    const int per_unit = p.n_row_tiles * p.n_split;
    it.unit = item / per_unit;
    const int rem = item - it.unit * per_unit;
    it.tile = rem / p.n_split;
    it.split = rem - it.tile * p.n_split;
    it.g0 = it.split * p.groups_per_split;
    it.g1 = min(p.L.n_groups, it.g0 + p.groups_per_split);
    return it;
}

// unsigned 8-bit x signed 8-bit -> int32, A and B K-major, M = 128
__device__ __forceinline__ uint32_t instr_desc_i8(int n) {
    return (2u << 4) | (0u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ void tc_mma_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld8(uint32_t taddr, uint32_t (&v)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "r"(taddr) : "memory");
}

// The GS codes of one segment of one row -> GS/4 operand cells (four unsigned bytes each, the code
// moved to bit P of its byte = its position inside the top-width code), written to TMEM columns
// [taddr, taddr + GS/4).  SW: storage width, W: logical width (W <= SW).
template <int GS, int SW>
__device__ __forceinline__ void unpack_segment(uint32_t seg, int rr, int W, int P, uint32_t taddr) {
    constexpr int ROW_BYTES = GS * SW / 8;
    constexpr int CS = ROW_BYTES < 16 ? ROW_BYTES : 16;      // chunk size of the packed layout
    constexpr int NLD = ROW_BYTES / CS;
    constexpr int WPL = CS / 4;                              // words per load
    constexpr int CPW = 8 / SW;                              // cells per word
    constexpr int NCELL = GS / 4;
    const uint32_t mask = (((1u << W) - 1u) << P) * 0x01010101u;

    constexpr int NB = NCELL / 8;                            // batches of 8 cells = one tcgen05.st (few live registers)
    constexpr int WPB = 8 / CPW;                             // words per batch: 4, 2, 1 for SW = 4, 2, 1 (8 for 8)
    constexpr int NW = NLD * WPL;
    // words are loaded batch by batch when a batch spans whole loads, otherwise once for all batches
    constexpr bool PER_BATCH = WPB >= WPL;
    uint32_t w[PER_BATCH ? WPB : NW];
    auto load = [&](int l, uint32_t* dst) {
        const uint32_t addr = seg + (uint32_t)((l * D2MOE_TILE_ROWS + rr) * CS);
        if constexpr (WPL == 4) {
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(dst[0]), "=r"(dst[1]), "=r"(dst[2]), "=r"(dst[3]) : "r"(addr));
        } else if constexpr (WPL == 2) {
            asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(dst[0]), "=r"(dst[1]) : "r"(addr));
        } else {
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(dst[0]) : "r"(addr));
        }
    };
    if constexpr (!PER_BATCH) {
#pragma unroll
        for (int l = 0; l < NLD; ++l) load(l, w + l * WPL);
    }
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        if constexpr (PER_BATCH) {
#pragma unroll
            for (int l = 0; l < WPB / WPL; ++l) load(b * (WPB / WPL) + l, w + l * WPL);
        }
        uint32_t v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int cell = b * 8 + i, q = PER_BATCH ? i / CPW : cell / CPW, u = cell % CPW;
            const int sh = P - SW * u;                       // compile-time sign when P is a constant
            const uint32_t moved = sh >= 0 ? (w[q] << (sh & 31)) : (w[q] >> ((-sh) & 31));
            v[i] = moved & mask;
        }
        tc_st8(taddr + b * 8, v);
    }
}

// Eight operand cells (batch b of a row's GS/4 cells) from one stored field of FW bits per code at bit PF of its
// byte; FIRST: the cells are set, otherwise the field is OR-ed into them (one three-input logic operation).
template <int GS, int FW, bool FIRST>
__device__ __forceinline__ void field_batch(uint32_t seg, int rr, int PF, int b, uint32_t (&v)[8]) {
    constexpr int ROW_BYTES = GS * FW / 8;
    constexpr int CS = ROW_BYTES < 16 ? ROW_BYTES : 16;
    constexpr int CPW = 8 / FW;                              // cells per word
    constexpr int WPB = FW;                                  // words per batch of 8 cells
    uint32_t w[WPB];
    auto addr_of = [&](int m) {                              // shared address of the row's word m
        const int ob = 4 * m, c = ob / CS, within = ob % CS;
        return seg + (uint32_t)((c * D2MOE_TILE_ROWS + rr) * CS + within);
    };
    if constexpr (WPB == 8) {
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(addr_of(8 * b)));
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]) : "r"(addr_of(8 * b + 4)));
    } else if constexpr (WPB == 4) {
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(addr_of(4 * b)));
    } else if constexpr (WPB == 2) {
        asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(w[0]), "=r"(w[1]) : "r"(addr_of(2 * b)));
    } else {
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w[0]) : "r"(addr_of(b)));
    }
    const uint32_t mask = (((1u << FW) - 1u) << PF) * 0x01010101u;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int q = i / CPW, u = i % CPW;
        const int sh = PF - FW * u;
        const uint32_t moved = sh >= 0 ? (w[q] << (sh & 31)) : (w[q] >> ((-sh) & 31));
        v[i] = FIRST ? (moved & mask) : ((moved & mask) | v[i]);
    }
}

// One width step of W bits (stored as fields of 8, 4, 2, 1 bits, widest first, one after the other in the block) of
// one row -> GS/4 operand cells with the step's value at bit P of every byte: the fields are merged in registers, so
// a step is one operand tile whatever its width.
template <int GS, int W>
__device__ __forceinline__ void unpack_step(uint32_t seg, int rr, int P, uint32_t taddr) {
    constexpr int F0 = W >= 8 ? 8 : (W >= 4 ? 4 : (W >= 2 ? 2 : 1));
    constexpr int R1 = W - F0;
    constexpr int F1 = R1 >= 4 ? 4 : (R1 >= 2 ? 2 : (R1 >= 1 ? 1 : 0));
    constexpr int R2 = R1 - F1;
    constexpr int F2 = R2 >= 2 ? 2 : (R2 >= 1 ? 1 : 0);
    constexpr int R3 = R2 - F2;                              // 0 or 1
    constexpr int FB = D2MOE_TILE_ROWS * GS / 8;             // bytes of a one-bit field
#pragma unroll
    for (int b = 0; b < GS / 32; ++b) {
        uint32_t v[8];
        field_batch<GS, F0, true>(seg, rr, P + R1, b, v);
        if constexpr (F1 > 0) field_batch<GS, F1, false>(seg + F0 * FB, rr, P + R2, b, v);
        if constexpr (F2 > 0) field_batch<GS, F2, false>(seg + (F0 + F1) * FB, rr, P + R3, b, v);
        if constexpr (R3 > 0) field_batch<GS, 1, false>(seg + (F0 + F1 + F2) * FB, rr, P, b, v);
        tc_st8(taddr + b * 8, v);
    }
}

template <int GS>
__device__ __forceinline__ void unpack_dispatch(int sw, uint32_t seg, int rr, int W, int P, uint32_t taddr) {
    switch (sw) {
        case 1: unpack_segment<GS, 1>(seg, rr, W, P, taddr); break;
        case 2: unpack_segment<GS, 2>(seg, rr, W, P, taddr); break;
        case 4: unpack_segment<GS, 4>(seg, rr, W, P, taddr); break;
        default: unpack_segment<GS, 8>(seg, rr, W, P, taddr); break;
    }
}

template <int WPACK> using I8SegList = WidthList<WPACK>;

// Output phase of one work item for one thread: scales the folded sums by the tokens' activation
// scales, applies SwiGLU across the gate / up rows of a hidden unit (mode 0) and writes the result.
// blks_lo / blks_hi: byte i = first slot / 4 of block i (blocks 0..3, 4..7).  rec: the warp's record of the work
// item in shared memory (words 0..31: activation scale of the unit's slots, copied asynchronously when the item
// began; 32: first slot, 33: tile, 34: split), so that the phase starts without a trip to global memory.
template <int NB>
static __device__ __noinline__ void i8_write_out(const I8Params& p, int r, int n_mine, uint32_t blks_lo, uint32_t blks_hi,
                                                 float (&acc)[NB][4], uint8_t* smem) {
    const float* rec = reinterpret_cast<const float*>(smem + p.smem_rec_off) + ((threadIdx.x >> 5) - 4) * 40;
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncwarp();
    const int slot0 = reinterpret_cast<const int*>(rec)[32];
    const int io_tile = reinterpret_cast<const int*>(rec)[33], io_split = reinterpret_cast<const int*>(rec)[34];
    const int blk = r & 1, rr = r >> 1;
    auto blk_of = [&](int i) -> uint32_t { return ((i < 4 ? blks_lo : blks_hi) >> (8 * (i & 3))) & 255u; };
#pragma unroll
    for (int i = 0; i < NB; ++i) {
        if (i < n_mine) {
            const float4 sg = *reinterpret_cast<const float4*>(rec + 4 * blk_of(i));
            acc[i][0] *= sg.x; acc[i][1] *= sg.y; acc[i][2] *= sg.z; acc[i][3] *= sg.w;
        }
    }
    if (p.mode == 0) {
        // lanes 2i and 2i + 1 hold the gate and the up row of hidden unit i of the tile: the two exchange by
        // shuffle so that each finishes half of the blocks (the gate lane the even blocks with the other's up
        // values, the up lane the odd blocks with the other's gate values)
#pragma unroll
        for (int i = 0; i < NB / 2; ++i) {
            if (2 * i < n_mine) {                                // uniform across the warp
                float other[4];
#pragma unroll
                for (int s = 0; s < 4; ++s)
                    other[s] = __shfl_xor_sync(0xffffffffu, blk == 0 ? acc[2 * i + 1][s] : acc[2 * i][s], 1);
                const int ib = 2 * i + blk;                      // the block this lane finishes
                if (ib < n_mine) {
                    float* dst = p.hbuf + (long long)(slot0 + 4 * blk_of(ib)) * p.D.F + (long long)io_tile * 64 + rr;
#pragma unroll
                    for (int s = 0; s < 4; ++s) {
                        const float g = blk == 0 ? acc[2 * i][s] : other[s];
                        const float up = blk == 0 ? other[s] : acc[2 * i + 1][s];
                        dst[(long long)s * p.D.F] = g / (1.0f + __expf(-g)) * up;
                    }
                }
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            if (i < n_mine) {
                float* dst = p.obuf + (long long)io_split * p.R_alloc * p.D.d
                           + (long long)(slot0 + 4 * blk_of(i)) * p.D.d + (long long)io_tile * 128 + blk * 64 + rr;
#pragma unroll
                for (int s = 0; s < 4; ++s) dst[(long long)s * p.D.d] = acc[i][s];
            }
        }
    }
}

template <int GS, int SWPACK, int NF>
__global__ void __launch_bounds__(i8_threads(NF), 2)
ffn_i8_kernel(const __grid_constant__ I8Params p, const __grid_constant__ TmaMaps maps) {
    constexpr int I8_WARP_PROD = 4 + 4 * NF, I8_WARP_MMA = 5 + 4 * NF;
    constexpr int NB = 8 / NF;                 // token blocks a fold warpgroup takes at most
    constexpr int GPS = 128 / GS;              // groups per ring stage (a stage spans 128 input columns)
    constexpr int KSTEPS = GS / 32;            // MMAs (K = 32) per segment and group
    extern __shared__ uint8_t smem_raw[];
    // shared layout from a 1024-byte boundary:
    // [activation tiles: I8_NSB x 8 KiB] [activation sums: I8_NSB x 512 B] [weight ring: nsw x GPS x 2 blocks] [work-item records] [barriers]
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t w_slot_bytes = (uint32_t)(GPS * 2) * (uint32_t)p.L.block_bytes;
    const uint32_t bbuf = smem_base;
    const uint32_t xkbuf = smem_base + I8_NSB * I8_B_TILE;   // per stage: 2 x (X, kappa) of 32 slots
    const uint32_t wbuf = smem_base + p.smem_w_off;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.smem_bar_off);
    const uint32_t bar0 = smem_u32(bars);
    auto W_FULL = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    auto W_EMPTY = [&](int i) { return bar0 + 8u * (uint32_t)(I8_MAX_NSW + i); };
    auto B_FULL = [&](int i) { return bar0 + 8u * (uint32_t)(2 * I8_MAX_NSW + i); };
    auto B_EMPTY = [&](int i) { return bar0 + 8u * (uint32_t)(2 * I8_MAX_NSW + I8_NSB + i); };
    auto A_FULL = [&](int wg, int sl) { return bar0 + 8u * (uint32_t)(2 * I8_MAX_NSW + 2 * I8_NSB + wg * 2 + sl); };
    auto A_EMPTY = [&](int wg, int sl) { return bar0 + 8u * (uint32_t)(2 * I8_MAX_NSW + 2 * I8_NSB + 4 + wg * 2 + sl); };
    auto D_FULL = [&](int b) { return bar0 + 8u * (uint32_t)(2 * I8_MAX_NSW + 2 * I8_NSB + 8 + b); };
    auto D_EMPTY = [&](int b) { return bar0 + 8u * (uint32_t)(2 * I8_MAX_NSW + 2 * I8_NSB + 10 + b); };
    auto SQ_FULL = [&](int i) { return bar0 + 8u * (uint32_t)(2 * I8_MAX_NSW + 2 * I8_NSB + 12 + i); };
    auto SQ_EMPTY = [&](int i) { return bar0 + 8u * (uint32_t)(2 * I8_MAX_NSW + 2 * I8_NSB + 12 + I8_NSQ + i); };
    static_assert(8 * I8_N_BARS + 8 * I8_NSQ <= 488, "barrier block");
    // work queue entries (after the barriers): the producer takes work items from a global counter and
    // publishes them here, so that CTAs that drew cheap items take more of them
    volatile int* sq_item = reinterpret_cast<volatile int*>(reinterpret_cast<uint8_t*>(bars) + 8 * I8_N_BARS);
    // ... and with every entry the item's last operand (kmax of its unit), which the unpack warps need before they can
    // start: the producer reads the unit one item ahead, so they start without a trip to global memory
    volatile int* sq_kmax = sq_item + I8_NSQ;
    // ... and the slots each operand's product covers (npad of the unit), which the issuer needs (after the fold warps' records)
    volatile int* sq_npad = reinterpret_cast<volatile int*>(smem + p.smem_rec_off + 8 * 40 * 4);
    // tail of the 512-byte barrier block: TMEM base (488), device-status pointer (496), abort flag (504)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(bars) + 488);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(reinterpret_cast<uint8_t*>(bars) + 504);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < I8_MAX_NSW; ++i) { mbar_init(W_FULL(i), 1); mbar_init(W_EMPTY(i), 4 + 4 * NF); }
        // an activation stage is released by the MMA issuer (its products have read the tile) and by
        // the fold warps (they have read the sums)
        for (int i = 0; i < I8_NSB; ++i) { mbar_init(B_FULL(i), 1); mbar_init(B_EMPTY(i), 1 + 4 * NF); }
        for (int wg = 0; wg < 2; ++wg)
            for (int sl = 0; sl < 2; ++sl) { mbar_init(A_FULL(wg, sl), 4); mbar_init(A_EMPTY(wg, sl), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(D_FULL(b), 1); mbar_init(D_EMPTY(b), 4 * NF); }
        // a queue entry is released by the issuer warp, the four unpack warps and the fold warps
        for (int i = 0; i < I8_NSQ; ++i) { mbar_init(SQ_FULL(i), 1); mbar_init(SQ_EMPTY(i), 5 + 4 * NF); }
        *abort_flag = 0;
        *reinterpret_cast<int32_t**>(reinterpret_cast<uint8_t*>(bars) + 496) = p.status;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == I8_WARP_MMA) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(I8_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t d_tmem = tmem_base;                         // buffer b: columns [64 b, 64 b + 64)
    const uint32_t a_tmem = tmem_base + 2 * I8_D_COLS;         // warpgroup wg, slot sl: + (wg*2 + sl)*32

    // set-up done (barriers, TMEM): from here on the kernel reads what the kernels before it wrote
    pdl_wait();
    const int n_units = *p.n_units;
    const int total_items = n_units * p.n_row_tiles * p.n_split;
    const int nsw = p.nsw;

    if (warp == I8_WARP_PROD) {
        // One producer thread feeds both rings, stage by stage (they are consumed at the same rate).
        if (lane == 0) {
            // This thread shares a scheduler with unpack warps, so its loop is kept short: source pointers and
            // ring positions advance by addition, nothing is recomputed per stage.
            uint32_t it = 0, ws = 0, wph = 1, bs = 0, bph = 1;         // ring positions, parity of the "empty" waits
            int item = blockIdx.x;
            // the fields of the item's unit that this thread needs, read one item ahead
            int u_e = 0, u_kmax = 0, u_nslots = 0, u_slot0 = 0, u_npad[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            if (item < total_items) {
                const I8Unit* u0 = p.units + i8_item(p, item).unit;
                u_e = u0->e; u_kmax = u0->kmax; u_nslots = u0->nslots; u_slot0 = u0->slot0;
#pragma unroll
                for (int j = 0; j < 8; ++j) u_npad[j] = u0->npad[j];
            }
            for (uint32_t qi = 0;; ++qi) {
                const uint32_t q = qi & (I8_NSQ - 1);
                mbar_wait_blk(SQ_EMPTY(q), ((qi / I8_NSQ) & 1u) ^ 1u);
                if (item >= total_items) item = -1;                    // the end mark
                sq_item[q] = item;
                sq_kmax[q] = u_kmax;
#pragma unroll
                for (int j = 0; j < 8; ++j) sq_npad[8 * q + j] = u_npad[j];
                mbar_arrive(SQ_FULL(q));
                if (item < 0) break;
                const int next = atomicAdd(p.next_item, 1);            // in flight while this item's stages are issued
                const I8Item ii = i8_item(p, item);
                const int e = u_e, kmax = u_kmax;
                // kmax: the unit's last width step (specialised kernels: a step is one operand) or its last stored segment
                const uint32_t bytes = (uint32_t)(SWPACK != 0 ? d2moe_prefix_bytes(p.L, kmax) : p.L.seg_off[kmax + 1]);
                const uint8_t *m0, *m1;
                if (p.mode == 0) {
                    m0 = p.P.w[3 * e + 0] + d2moe_block_offset(p.L, ii.tile, ii.g0);
                    m1 = p.P.w[3 * e + 1] + d2moe_block_offset(p.L, ii.tile, ii.g0);
                } else {
                    m0 = p.P.w[3 * e + 2] + d2moe_block_offset(p.L, 2 * ii.tile, ii.g0);
                    m1 = p.P.w[3 * e + 2] + d2moe_block_offset(p.L, 2 * ii.tile + 1, ii.g0);
                }
                const int nslots = u_nslots, slot0 = u_slot0;
                const int mi = nslots <= 8 ? 0 : (nslots <= 16 ? 1 : 2);        // boxes of 16, 32, 64 rows
                const uint32_t tile_bytes = (16u << mi) * 128u;
                const uint32_t xk_bytes = (uint32_t)nslots * 8u;
                const uint32_t bb = (uint32_t)p.L.block_bytes;
                const float* xk_src = p.xk + ((long long)ii.g0 * p.R_alloc + slot0) * 2;
                const long long xk_step = p.R_alloc * 2;
                const CUtensorMap* map = &maps.m[mi];
                if (next < total_items) {                              // the next item's unit: in flight during the stage loop
                    const I8Unit* un = p.units + i8_item(p, next).unit;
                    u_e = un->e; u_kmax = un->kmax; u_nslots = un->nslots; u_slot0 = un->slot0;
#pragma unroll
                    for (int j = 0; j < 8; ++j) u_npad[j] = un->npad[j];
                }
                for (int G = ii.g0; G < ii.g1; G += GPS, ++it) {
                    const int ng = min(GPS, ii.g1 - G);
                    {
                        mbar_wait_blk(W_EMPTY(ws), wph);
                        mbar_expect_tx(W_FULL(ws), 2 * bytes * ng);
                        const uint32_t dst = wbuf + ws * w_slot_bytes;
#pragma unroll
                        for (int sub = 0; sub < GPS; ++sub) {
                            if (sub < ng) {
                                bulk_g2s(dst + (2 * sub) * bb, m0, bytes, W_FULL(ws));
                                bulk_g2s(dst + (2 * sub + 1) * bb, m1, bytes, W_FULL(ws));
                                m0 += bb; m1 += bb;
                            }
                        }
                        if (++ws == (uint32_t)nsw) { ws = 0; wph ^= 1u; }
                    }
                    {
                        mbar_wait_blk(B_EMPTY(bs), bph);
                        mbar_expect_tx(B_FULL(bs), tile_bytes + ng * xk_bytes);
                        tma_load_2d(bbuf + bs * I8_B_TILE, map, G * GS, 2 * slot0, B_FULL(bs));
#pragma unroll
                        for (int sub = 0; sub < GPS; ++sub) {
                            if (sub < ng) {
                                bulk_g2s(xkbuf + (2 * bs + sub) * I8_XK_BYTES, xk_src, xk_bytes, B_FULL(bs));
                                xk_src += xk_step;
                            }
                        }
                        if (++bs == I8_NSB) { bs = 0; bph ^= 1u; }
                    }
                }
                item = next;
            }
            for (int s = 0; s < nsw && s < (int)it; ++s) {      // drain: all copies issued have landed
                const uint32_t last = it - 1 - (it - 1 - s) % nsw;
                mbar_wait(W_FULL(s), (last / nsw) & 1, abort_flag, p.status, true);
            }
            for (int s = 0; s < I8_NSB && s < (int)it; ++s) {
                const uint32_t last = it - 1 - (it - 1 - s) % I8_NSB;
                mbar_wait(B_FULL(s), (last / I8_NSB) & 1, abort_flag, p.status, true);
            }
        }
    } else if (warp == I8_WARP_MMA) {
        // One issuer: all segments of a group accumulate into the same columns, so their products
        // must be issued in order.  The whole warp runs the loop and one elected lane issues, so that
        // addresses and descriptors stay in the uniform datapath.  A warpgroup hands over up to two
        // operand tiles at a time (its segments j and j + 2).
        uint32_t gc = 0, bs = 0, bph = 0, hs[2] = {0, 0};
        for (uint32_t qi = 0;; ++qi) {
            const uint32_t q = qi & (I8_NSQ - 1);
            mbar_wait_blk(SQ_FULL(q), (qi / I8_NSQ) & 1u);
            const int item = sq_item[q];
            const int kmax = sq_kmax[q];
            uint32_t idesc[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) idesc[j] = instr_desc_i8(2 * max(sq_npad[8 * q + j], 8));
            __syncwarp();                                       // the entry is released after its last read
            if (lane == 0) mbar_arrive(SQ_EMPTY(q));
            if (item < 0) break;
            const I8Item ii = i8_item(p, item);
            for (int G = ii.g0; G < ii.g1; G += GPS) {
                const int ng = min(GPS, ii.g1 - G);
                mbar_wait_blk(B_FULL(bs), bph);
                const uint64_t bdesc = smem_desc_sw128(bbuf + bs * I8_B_TILE);
#pragma unroll
                for (int sub = 0; sub < GPS; ++sub) {
                    if (sub < ng) {
                        const int buf = gc & 1;
                        mbar_wait_blk(D_EMPTY(buf), ((gc >> 1) & 1) ^ 1);
                        tc_fence_after();
                        const uint32_t d_addr = d_tmem + buf * I8_D_COLS;
#pragma unroll
                        for (int hp = 0; hp < (SWPACK != 0 ? (I8SegList<SWPACK>::count() + 3) / 4 : 2); ++hp) {
#pragma unroll
                            for (int wg = 0; wg < 2; ++wg) {
                                const int j0 = wg + 4 * hp, j1 = j0 + 2;
                                if (j0 <= kmax) {
                                    mbar_wait_blk(A_FULL(wg, 0), hs[wg] & 1);
                                    tc_fence_after();
                                    const uint32_t a_addr = a_tmem + wg * 64;
                                    if (elect_one()) {
#pragma unroll
                                        for (int ks = 0; ks < KSTEPS; ++ks)
                                            tc_mma_i8_ts(d_addr, a_addr + ks * 8, bdesc + (uint64_t)((sub * GS + ks * 32) >> 4),
                                                         idesc[j0], (j0 == 0 && ks == 0) ? 0u : 1u);
                                        if (j1 <= kmax) {
#pragma unroll
                                            for (int ks = 0; ks < KSTEPS; ++ks)
                                                tc_mma_i8_ts(d_addr, a_addr + 32 + ks * 8, bdesc + (uint64_t)((sub * GS + ks * 32) >> 4),
                                                             idesc[j1 & 7], 1u);
                                        }
                                        tc_commit(A_EMPTY(wg, 0));
                                    }
                                    __syncwarp();
                                    ++hs[wg];
                                }
                            }
                        }
                        if (elect_one()) tc_commit(D_FULL(buf));
                        __syncwarp();
                        ++gc;
                    }
                }
                if (elect_one()) tc_commit(B_EMPTY(bs));
                __syncwarp();
                if (++bs == I8_NSB) { bs = 0; bph ^= 1; }
            }
        }
        // all products have completed before TMEM is released
        if (gc > 0) mbar_wait(D_FULL((gc - 1) & 1), ((gc - 1) >> 1) & 1, abort_flag, p.status, true);
        if (gc > 1) mbar_wait(D_FULL((gc - 2) & 1), ((gc - 2) >> 1) & 1, abort_flag, p.status, true);
    } else if (warp < 4) {
        // -------- unpack warpgroup: fills both operand slots of every group (slot 0: segments 0, 2, (4, 6); slot 1:
        // segments 1, 3, (5, 7)), one hand-off per slot --------
        const int r = threadIdx.x & 127;           // row of the tile = TMEM lane
        const int blk = r & 1, rr = r >> 1;         // lanes 2i, 2i + 1: row i of the tile's two packed blocks
        const uint32_t lane_addr = ((uint32_t)((warp & 3) * 32)) << 16;
        uint32_t hs[2] = {0, 0};                   // hand-offs so far, per slot
        uint32_t ws = 0, wph = 0;
        uint32_t w_addr = wbuf + (uint32_t)blk * (uint32_t)p.L.block_bytes;
        for (uint32_t qi = 0;; ++qi) {
            const uint32_t q = qi & (I8_NSQ - 1);
            mbar_wait_blk(SQ_FULL(q), (qi / I8_NSQ) & 1u);
            const int item = sq_item[q];
            const int kmax = sq_kmax[q];
            __syncwarp();
            if (lane == 0) mbar_arrive(SQ_EMPTY(q));
            if (item < 0) break;
            const I8Item ii = i8_item(p, item);
            for (int G = ii.g0; G < ii.g1; G += GPS) {
                const int ng = min(GPS, ii.g1 - G);
                mbar_wait_blk(W_FULL(ws), wph);
#pragma unroll
                for (int sub = 0; sub < GPS; ++sub) {
                    if (sub < ng) {
                        const uint32_t wb = w_addr + (uint32_t)(2 * sub) * (uint32_t)p.L.block_bytes;
                        auto handoff_begin = [&](int sl) {
                            mbar_wait_blk(A_EMPTY(sl, 0), (hs[sl] & 1) ^ 1);
                            tc_fence_after();
                        };
                        auto handoff_end = [&](int sl) {
                            tc_wait_st();
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(A_FULL(sl, 0));
                            ++hs[sl];
                        };
                        if constexpr (SWPACK != 0) {
                            using SL = I8SegList<SWPACK>;
                            auto do_seg = [&](auto jc) {
                                constexpr int J = decltype(jc)::value;
                                if constexpr (J < SL::count()) {
                                    if (J <= kmax) {
                                        const uint32_t taddr = a_tmem + (J & 1) * 64 + lane_addr + ((J >> 1) & 1) * 32;
                                        if constexpr (SL::w(J) == SL::sw(J))
                                            unpack_segment<GS, SL::sw(J)>(wb + (uint32_t)SL::seg_off(GS, J), rr, SL::w(J), SL::pos(J), taddr);
                                        else
                                            unpack_step<GS, SL::w(J)>(wb + (uint32_t)SL::seg_off(GS, J), rr, SL::pos(J), taddr);
                                    }
                                }
                            };
                            constexpr int NHP = (SL::count() + 3) / 4;
                            {                                        // slot 0: segments 0, 2
                                handoff_begin(0);
                                do_seg(std::integral_constant<int, 0>{});
                                do_seg(std::integral_constant<int, 2>{});
                                handoff_end(0);
                            }
                            if (1 <= kmax) {                         // slot 1: segments 1, 3
                                handoff_begin(1);
                                do_seg(std::integral_constant<int, 1>{});
                                do_seg(std::integral_constant<int, 3>{});
                                handoff_end(1);
                            }
                            if constexpr (NHP > 1) {
                                if (4 <= kmax) {
                                    handoff_begin(0);
                                    do_seg(std::integral_constant<int, 4>{});
                                    do_seg(std::integral_constant<int, 6>{});
                                    handoff_end(0);
                                }
                                if (5 <= kmax) {
                                    handoff_begin(1);
                                    do_seg(std::integral_constant<int, 5>{});
                                    do_seg(std::integral_constant<int, 7>{});
                                    handoff_end(1);
                                }
                            }
                        } else {
#pragma unroll 1
                            for (int j0 = 0; j0 <= kmax; j0 += 4) {
#pragma unroll 1
                                for (int sl = 0; sl < 2; ++sl) {
                                    const int j = j0 + sl;
                                    if (j > kmax) break;
                                    const uint32_t taddr = a_tmem + sl * 64 + lane_addr;
                                    handoff_begin(sl);
                                    unpack_dispatch<GS>(p.L.seg_sw[j], wb + (uint32_t)p.L.seg_off[j], rr, p.L.seg_w[j], p.L.seg_shift[j], taddr);
                                    if (j + 2 <= kmax)
                                        unpack_dispatch<GS>(p.L.seg_sw[j + 2], wb + (uint32_t)p.L.seg_off[j + 2], rr, p.L.seg_w[j + 2],
                                                            p.L.seg_shift[j + 2], taddr + 32);
                                    handoff_end(sl);
                                }
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(W_EMPTY(ws));
                w_addr += w_slot_bytes;
                if (++ws == (uint32_t)nsw) { ws = 0; wph ^= 1; w_addr = wbuf + (uint32_t)blk * (uint32_t)p.L.block_bytes; }
            }
        }
    } else if (warp < 4 + 4 * NF) {
        // -------- the fold warpgroups: every group's accumulator into fp32 sums; with two warpgroups each takes half of the
        // unit's token blocks (at most 4), one takes all (at most 8); output phase --------
        const int wg = (warp >> 2) - 1;            // 0 .. NF - 1
        const int r = threadIdx.x & 127;           // row of the tile = TMEM lane
        const int blk = r & 1, rr = r >> 1;         // lanes 2i, 2i + 1: row i of the tile's two packed blocks
        const uint32_t lane_addr = ((uint32_t)((warp & 3) * 32)) << 16;
        const uint32_t d_base = d_tmem + lane_addr;
        uint32_t gc = 0;                           // groups folded so far
        uint32_t ws = 0, bs = 0;                   // ring positions
        uint32_t w_addr = wbuf + (uint32_t)blk * (uint32_t)p.L.block_bytes;
        const float s1_factor = __int_as_float((127 - (p.L.top - p.L.b1)) << 23);
        for (uint32_t qi = 0;; ++qi) {
            const uint32_t q = qi & (I8_NSQ - 1);
            mbar_wait_blk(SQ_FULL(q), (qi / I8_NSQ) & 1u);
            const int item = sq_item[q];
            __syncwarp();
            if (lane == 0) mbar_arrive(SQ_EMPTY(q));
            if (item < 0) break;
            const I8Item ii = i8_item(p, item);
            const I8Unit* u = p.units + ii.unit;
            const int nblk = u->nblk;
            {
                float* rec = reinterpret_cast<float*>(smem + p.smem_rec_off) + (warp - 4) * 40;     // this warp's record of the item
                const int slot0 = u->slot0;
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4;"
                             ::"r"(smem_u32(rec + lane)), "l"(p.sigma + slot0 + lane) : "memory");
                asm volatile("cp.async.commit_group;" ::: "memory");
                if (lane == 0) {
                    reinterpret_cast<int*>(rec)[32] = slot0;
                    reinterpret_cast<int*>(rec)[33] = ii.tile;
                    reinterpret_cast<int*>(rec)[34] = ii.split;
                }
            }
            const int h0 = (nblk + 1) >> 1;
            const int f0 = (NF == 2 && wg == 1) ? h0 : 0;        // my first block
            const int n_mine = NF == 2 ? (wg == 0 ? h0 : nblk - h0) : nblk;     // my token blocks (at most NB)
            uint32_t myblks[2] = {0, 0};                         // byte i of word i / 4: first slot / 4 of my block i
#pragma unroll
            for (int i = 0; i < NB; ++i) myblks[i >> 2] |= (uint32_t)u->blk[min(f0 + i, 7)] << (8 * (i & 3));
            uint32_t blk_r[NB];
#pragma unroll
            for (int i = 0; i < NB; ++i) blk_r[i] = (myblks[i >> 2] >> (8 * (i & 3))) & 255u;
            // the round (of two blocks) after whose loads the accumulator is released: with one fold warpgroup the last
            // one that loads anything (up to four rounds), with two always the second (a warpgroup without blocks of
            // its own still releases)
            const int last_rd = NF == 1 ? (n_mine > 0 ? (n_mine - 1) >> 1 : 0) : NB / 2 - 1;
            float acc[NB][4];
#pragma unroll
            for (int i = 0; i < NB; ++i)
#pragma unroll
                for (int s = 0; s < 4; ++s) acc[i][s] = 0.0f;

            for (int G = ii.g0; G < ii.g1; G += GPS) {
                const int ng = min(GPS, ii.g1 - G);
                // The fold waits for one thing only, the finished accumulator of a group: its products were issued after
                // the issuer had seen the stage's activation tile arrive and after the unpack warps had seen the stage's
                // packed blocks arrive, so both are in shared memory by then (the fold still releases both stages: they are
                // not refilled before it has read its part of them).
                uint32_t meta[GPS];
#pragma unroll
                for (int sub = 0; sub < GPS; ++sub) {
                    if (sub < ng) {
                        const int buf = gc & 1;
                        mbar_wait_blk(D_FULL(buf), (gc >> 1) & 1);
                        tc_fence_after();
                        if (sub == 0) {
                            // the scales of this stage's groups, then the stage is released as far as this warp goes
#pragma unroll
                            for (int s2 = 0; s2 < GPS; ++s2)
                                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(meta[s2])
                                             : "r"(w_addr + (uint32_t)(2 * s2) * (uint32_t)p.L.block_bytes + 4u * rr));
                            __syncwarp();
                            if (lane == 0) mbar_arrive(W_EMPTY(ws));
                            w_addr += w_slot_bytes;
                            if (++ws == (uint32_t)nsw) { ws = 0; w_addr = wbuf + (uint32_t)blk * (uint32_t)p.L.block_bytes; }
                        }
                        const __half2 mh = as_h2(meta[sub]);
                        const float s1p = __low2float(mh) * s1_factor;
                        const float lo = __high2float(mh);
                        const uint32_t xk_addr = xkbuf + (bs * 2 + sub) * I8_XK_BYTES;
                        const uint32_t d_addr = d_base + buf * I8_D_COLS;
                        auto fold_block = [&](int b, const uint32_t (&v)[8]) {
                            float xk[8];
                            const uint32_t a = xk_addr + 32u * blk_r[b];
                            asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(xk[0]), "=f"(xk[1]), "=f"(xk[2]), "=f"(xk[3]) : "r"(a));
                            asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(xk[4]), "=f"(xk[5]), "=f"(xk[6]), "=f"(xk[7]) : "r"(a + 16u));
                            const float cx = fmaf(s1p, xk[1], lo);
#pragma unroll
                            for (int s = 0; s < 4; ++s) {
                                const int di = (int)v[2 * s] * 128 + (int)v[2 * s + 1];
                                acc[b][s] = fmaf(s1p, (float)di, acc[b][s]);
                                acc[b][s] = fmaf(cx, xk[2 * s], acc[b][s]);
                            }
                        };
                        // rounds of two blocks, one set of loaded values at a time (registers); the accumulator is released
                        // as soon as the last round's values are in registers
#pragma unroll
                        for (int rd = 0; rd < NB / 2; ++rd) {
                            if (rd <= last_rd) {
                                uint32_t v[2][8];
#pragma unroll
                                for (int i = 0; i < 2; ++i)
                                    if (2 * rd + i < n_mine) tc_ld8(d_addr + 8 * blk_r[2 * rd + i], v[i]);
                                tc_wait_ld();
                                if (rd == last_rd) { tc_fence_before(); __syncwarp(); if (lane == 0) mbar_arrive(D_EMPTY(buf)); }
#pragma unroll
                                for (int i = 0; i < 2; ++i)
                                    if (2 * rd + i < n_mine) fold_block(2 * rd + i, v[i]);
                            }
                        }
                        ++gc;
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(B_EMPTY(bs));
                if (++bs == I8_NSB) bs = 0;
            }

            // ---- write out: y = sigma * acc (out of line: its registers are not the loop's) ----
            float out[NB][4];                  // a copy: acc itself must stay in registers
#pragma unroll
            for (int i = 0; i < NB; ++i)
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) out[i][q4] = acc[i][q4];
            i8_write_out<NB>(p, r, n_mine, myblks[0], myblks[1], out, smem);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == I8_WARP_MMA) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(I8_TMEM_COLS) : "memory");
    }
}

__device__ __forceinline__ int round8(int n) { return (n + 7) & ~7; }

// One block.  Lays every expert's tokens out by width, widest first, each width class padded to a
// multiple of 8 slots; cuts every expert into units of 32 slots; records per unit and segment how many
// of its slots include the segment, and which blocks of 4 slots hold real tokens.
// Then orders the units by decreasing work per group, so that the expert kernels, whose CTAs draw work
// items from a counter, take the cheap ones last; sets both work counters (n_units[1], n_units[2]) to
// the grid size of those kernels.
// Shared memory: group_off (E K + 1 ints), per expert its first unit (n_exp + 1 ints), per unit its cost (max_units ints),
// the padded slot offsets (n_exp + 1 ints).
__global__ void __launch_bounds__(512)
i8_prep_kernel(MoeDims D, RouteBufs R, I8Unit* units, int* n_units, int32_t* pad_off, int32_t* row_map,
               int32_t* src_token, float* kappa, int max_units, int top, int b1, int ffn_grid, int32_t* status,
               I8SegMap sm, const int32_t* group_keys) {
    pdl_enter();
    extern __shared__ int32_t s_prep[];
    // decode-sized loads: the grouping of the assignments by (expert, width) first, in this launch (the routing
    // kernels left it to this one); its results are read below after a barrier, by this same block
    if (group_keys) {
        if (d2moe_group_is_sortable(D.A, D.E * D.K)) group_sort_body(D.A, D.E * D.K, group_keys, R.group_off, R.perm, R.inv_perm, s_prep);
        else group_block_body(D.A, D.E * D.K, group_keys, R.group_off, R.perm, R.inv_perm, s_prep, 0, 1);
        __syncthreads();
    }
    __shared__ int s_total;
    const int n_exp = D.E + D.n_shared, n_keys = D.E * D.K;
    int32_t* go = s_prep;                          // group_off
    int32_t* unit_off = s_prep + n_keys + 1;
    int32_t* cost = unit_off + n_exp + 1;
    int32_t* s_pad = cost + max_units;             // pad_off, kept here too (read back below without a trip to global memory)
    for (int i = threadIdx.x; i <= n_keys; i += blockDim.x) go[i] = R.group_off[i];
    __syncthreads();
    if (threadIdx.x < 32) {                       // padded slot offsets and first units (one warp scans)
        const int lane = threadIdx.x;
        int carry = 0, ucarry = 0;
        for (int base = 0; base < n_exp; base += 32) {
            const int e = base + lane;
            int v = 0;
            if (e < D.E) {
                for (int j = 0; j < D.K; ++j) v += round8(go[e * D.K + j + 1] - go[e * D.K + j]);
            } else if (e < n_exp) {
                v = round8(D.T);
            }
            const int nu = (v + I8_SLOTS - 1) / I8_SLOTS;
            int incl = v, uincl = nu;
            for (int off = 1; off < 32; off <<= 1) {
                const int o = __shfl_up_sync(0xffffffffu, incl, off);
                const int uo = __shfl_up_sync(0xffffffffu, uincl, off);
                if (lane >= off) { incl += o; uincl += uo; }
            }
            if (e < n_exp) { pad_off[e] = carry + incl - v; s_pad[e] = carry + incl - v; unit_off[e] = ucarry + uincl - nu; }
            carry += __shfl_sync(0xffffffffu, incl, 31);
            ucarry += __shfl_sync(0xffffffffu, uincl, 31);
        }
        if (lane == 0) {
            pad_off[n_exp] = carry; s_pad[n_exp] = carry; s_total = carry; unit_off[n_exp] = ucarry;
            n_units[0] = min(ucarry, max_units);
            n_units[1] = ffn_grid; n_units[2] = ffn_grid;
        }
    }
    __syncthreads();
    const int total = s_total;
    for (int i = threadIdx.x; i < total; i += blockDim.x) { src_token[i] = -1; kappa[i] = 0.0f; }
    __syncthreads();
    for (int a = threadIdx.x; a < D.A; a += blockDim.x) {
        const int pos = R.inv_perm[a];
        const int e = R.topk_idx[a], kk = R.bit_idx[a];
        // a supplied routing index out of range: the assignment is skipped (row -1 contributes nothing to the
        // combine; its slot stays a padding slot) and the call is flagged
        if (e < 0 || e >= D.E || kk < 0 || kk >= D.K || pos < 0 || pos >= D.A) {
            row_map[a] = -1;
            if (status) atomicOr(status, D2MOE_DEV_BAD_INDEX);
            continue;
        }
        int start = 0;                            // classes of a larger width index come first
        for (int i = kk + 1; i < D.K; ++i) start += round8(go[e * D.K + i + 1] - go[e * D.K + i]);
        const int slot = s_pad[e] + start + (pos - go[e * D.K + kk]);
        // pos must lie inside the group of (e, kk); otherwise the permutation does not belong to these indices
        if (pos < go[e * D.K + kk] || pos >= go[e * D.K + kk + 1] || slot < 0 || slot >= total) {
            row_map[a] = -1;
            if (status) atomicOr(status, D2MOE_DEV_BAD_INDEX);
            continue;
        }
        row_map[a] = slot;
        src_token[slot] = a / D.k;
        kappa[slot] = exp2f((float)(top - D.bits[kk] - 1)) - exp2f((float)(top - b1 - 1));
    }
    for (int i = threadIdx.x; i < D.n_shared * D.T; i += blockDim.x) {
        const int s = i / D.T, t = i - s * D.T;
        const int slot = s_pad[D.E + s] + t;
        row_map[D.A + i] = slot;
        src_token[slot] = t;
        kappa[slot] = 0.5f - exp2f((float)(top - b1 - 1));
    }
    // one thread per unit (an expert with many tokens, a shared one above all, has many units): the unit's
    // expert is the last one whose first unit is not beyond it
    const int n_all = min(unit_off[n_exp], max_units);
    I8Unit mine[4];                               // this thread's first four units stay in registers for the ordering below
    for (int nu = threadIdx.x, mk = 0; nu < n_all; nu += blockDim.x, ++mk) {
        int lo_e = 0, hi_e = n_exp - 1;
        while (lo_e < hi_e) {
            const int mid = (lo_e + hi_e + 1) >> 1;
            if (unit_off[mid] <= nu) lo_e = mid; else hi_e = mid - 1;
        }
        while (lo_e + 1 < n_exp && unit_off[lo_e + 1] <= nu) ++lo_e;       // skip experts without units
        const int e = lo_e;
        const int p0 = s_pad[e], len_e = s_pad[e + 1] - p0;
        int cnt[8], cpad[9];                      // cpad[j]: padded slots of the classes with index >= j
        cpad[D.K] = 0;
        for (int j = D.K - 1; j >= 0; --j) {
            cnt[j] = e < D.E ? go[e * D.K + j + 1] - go[e * D.K + j] : (j == D.K - 1 ? D.T : 0);
            cpad[j] = cpad[j + 1] + round8(cnt[j]);
        }
        {
            const int start = (nu - unit_off[e]) * I8_SLOTS;
            const int len = min(len_e - start, I8_SLOTS);
            I8Unit u;
            u.e = e; u.slot0 = p0 + start; u.nslots = len; u.kmax = 0; u.nblk = 0;
            for (int j = 0; j < 8; ++j) {          // per stored segment: the slots of the width classes that include it
                u.blk[j] = 0;
                u.npad[j] = j < sm.n_seg ? max(0, min(len, cpad[sm.seg_kk[j]] - start)) : 0;
                if (u.npad[j] > 0) u.kmax = j;
            }
            for (int j = D.K - 1; j >= 0; --j) {          // real slots of class j: [cpad[j+1], cpad[j+1] + cnt[j])
                const int a0 = max(cpad[j + 1], start), a1 = min(cpad[j + 1] + cnt[j], start + len);
                for (int b = a0 / 4; 4 * b < a1; ++b)
                    if (u.nblk < 8) u.blk[u.nblk++] = b - start / 4;
            }
            // every window starts with a real token: never empty.  With few units the list is ordered below and
            // written then; otherwise it is written here, in the order it was built
            if (n_all > 4 * (int)blockDim.x) units[nu] = u;
            else {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (mk == k) mine[k] = u;
            }
            // work per group: one warpgroup unpacks every operand, the fold warps take the blocks (half each when there are two warpgroups)
            cost[nu] = 80 * (u.kmax + 1) + 25 * ((u.nblk + 1) / 2);
        }
    }
    __syncthreads();
    const int n = min(unit_off[n_exp], max_units);
    if (n <= 4 * (int)blockDim.x) {              // rank by (cost descending, index ascending), then permute
        int rank[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int i = threadIdx.x + k * blockDim.x;
            rank[k] = -1;
            if (i < n) {
                const int c = cost[i];
                int rk = 0;
                for (int j = 0; j < n; ++j) rk += (cost[j] > c || (cost[j] == c && j < i)) ? 1 : 0;
                rank[k] = rk;
            }
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (rank[k] >= 0) units[rank[k]] = mine[k];
    }
}

// Quantises one activation row per slot to 15-bit integers xq = rint(x / sigma), sigma = max|x| / 16191,
// stored as two signed bytes per element (xq = 128 hi + lo8, lo8 in [-64, 63]) in rows 2 slot and
// 2 slot + 1 of q, in the byte order of the operand cells (elements k, k+2, k+1, k+3), and writes
// per group the integer sum X of the row's xq, and kappa of the slot.  GATHER: the row of slot s is
// x[src_token[s]] (bf16); otherwise it is row s of an fp32 buffer.  Padding slots become zeros.
// One block per slot at a time; a thread keeps its cells (four elements each; cell c = threadIdx.x + k blockDim.x,
// k < I8_QCPT) in registers between the maximum and the rounding, so a row of up to 16 blockDim.x elements is read
// once (a longer row goes round by round and is read twice).  blockDim.x is a multiple of 32: the 32 (or 16) cells of
// a group sit in one warp.
constexpr int I8_QCPT = 4;
template <bool GATHER>
__global__ void __launch_bounds__(1024)
i8_quant_kernel(int n, int g, long long R_alloc, const void* __restrict__ src, const int32_t* __restrict__ src_token,
                const int32_t* __restrict__ pad_off, int n_off, const float* __restrict__ kappa,
                int8_t* __restrict__ q, float* __restrict__ xk, float* __restrict__ sigma, int32_t* status) {
    pdl_enter();
    __shared__ uint32_t s_red[32];
    const int total = pad_off[n_off];
    const int n_cells = n / 4, cpg = g / 4;                 // cells per group: 16 or 32
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const int per_round = I8_QCPT * blockDim.x;
    const bool single = n_cells <= per_round;             // the whole row fits the block's registers
    for (int slot = blockIdx.x; slot < total; slot += gridDim.x) {
        const int t = src_token[slot];
        float v[I8_QCPT][4];
        // cells [base, base + I8_QCPT blockDim.x) of the row into v; returns the bits of their largest magnitude
        // (they order like unsigned integers, a NaN or an infinity above every finite value)
        auto load_round = [&](int base) -> uint32_t {
            uint32_t m = 0;
#pragma unroll
            for (int k = 0; k < I8_QCPT; ++k) {
                const int c = base + threadIdx.x + k * blockDim.x;
                v[k][0] = v[k][1] = v[k][2] = v[k][3] = 0.0f;
                if (c < n_cells) {
                    if (GATHER) {
                        const uint2 raw = reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(src) + (size_t)t * n)[c];
                        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
                        const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
                        v[k][0] = a.x; v[k][1] = a.y; v[k][2] = b.x; v[k][3] = b.y;
                    } else {
                        const float4 f = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(src) + (size_t)slot * n)[c];
                        v[k][0] = f.x; v[k][1] = f.y; v[k][2] = f.z; v[k][3] = f.w;
                    }
#pragma unroll
                    for (int i = 0; i < 4; ++i) m = max(m, __float_as_uint(fabsf(v[k][i])));
                }
            }
            return m;
        };
        uint32_t mbits = 0;
        if (t >= 0)
            for (int base = 0; base < n_cells; base += per_round) mbits = max(mbits, load_round(base));
        mbits = __reduce_max_sync(0xffffffffu, mbits);
        if (lane == 0) s_red[warp] = mbits;
        __syncthreads();
        mbits = lane < n_warps ? s_red[lane] : 0u;
        mbits = __reduce_max_sync(0xffffffffu, mbits);
        __syncthreads();                           // s_red is free for the next slot
        const float amax = __uint_as_float(mbits);
        const bool bad = !(amax < 3.0e38f);        // a NaN or an infinity in the row
        const bool live = t >= 0 && amax > 0.0f && !bad;
        // a row with a NaN or an infinity cannot be quantised: its outputs are zero and the call is flagged
        if (bad && threadIdx.x == 0 && status) atomicOr(status, D2MOE_DEV_NONFINITE);
        const float scale = live ? I8_XMAX / amax : 0.0f;
        const float kap = kappa[slot];
        if (threadIdx.x == 0) sigma[slot] = live ? amax / I8_XMAX : 0.0f;
        uint32_t* qh = reinterpret_cast<uint32_t*>(q + (size_t)(2 * slot) * n);
        uint32_t* ql = reinterpret_cast<uint32_t*>(q + (size_t)(2 * slot + 1) * n);
        for (int base = 0; base < n_cells; base += per_round) {
        if (!single && live) load_round(base);
#pragma unroll
        for (int k = 0; k < I8_QCPT; ++k) {
            const int c = base + threadIdx.x + k * blockDim.x;
            int sum = 0;
            if (c < n_cells) {
                uint32_t wh = 0, wl = 0;
                if (live) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        int xq = __float2int_rn(v[k][i] * scale);
                        xq = max(-16191, min(16191, xq));
                        const int lo8 = ((xq + 64) & 127) - 64;
                        const int hi = (xq - lo8) >> 7;
                        const int byte = ((i & 1) << 1) | (i >> 1);
                        wh |= (uint32_t)(hi & 255) << (8 * byte);
                        wl |= (uint32_t)(lo8 & 255) << (8 * byte);
                        sum += xq;
                    }
                }
                qh[c] = wh; ql[c] = wl;
            }
            for (int off = cpg >> 1; off; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
            if (c < n_cells && (c % cpg) == 0) {
                const int G = c / cpg;
                float2 o;
                o.x = (float)sum; o.y = kap;
                reinterpret_cast<float2*>(xk)[(size_t)G * R_alloc + slot] = o;
            }
        }
        }
    }
}

// tensor maps over a row-major byte matrix [rows, cols], 128-byte swizzle, boxes of 128 columns x 16/32/64 rows
static inline bool make_maps_u8_uncached(TmaMaps* maps, void* base, long long rows, long long cols) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return false;
    for (int i = 0; i < 3; ++i) {
        cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
        cuuint64_t strides[1] = {(cuuint64_t)cols};
        cuuint32_t box[2] = {128, (cuuint32_t)(16 << i)};
        cuuint32_t estr[2] = {1, 1};
        if (enc(&maps->m[i], CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return false;
    }
    maps->m[3] = maps->m[2]; maps->m[4] = maps->m[2];
    return true;
}
static inline bool make_maps_u8(TmaMaps* maps, void* base, long long rows, long long cols) {
    return cached_maps(maps, 1, base, rows, cols, [&](TmaMaps* m) { return make_maps_u8_uncached(m, base, rows, cols); });
}

// One block waits on a barrier that nothing completes, with either of the two bounded waits of the
// expert kernels; the barrier block has the layout those waits expect (status pointer at byte 496, abort
// flag at byte 504 of a 512-byte aligned block).  A second wait follows: with the abort flag set it
// returns at once.
__global__ void __launch_bounds__(64)
wait_expiry_kernel(int which, int32_t* status) {
    __shared__ __align__(1024) uint8_t blk[1024];
    uint8_t* b = blk + ((512u - (smem_u32(blk) & 511u)) & 511u);
    const uint32_t bar = smem_u32(b);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(b + 504);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        *abort_flag = 0;
        *reinterpret_cast<int32_t**>(b + 496) = status;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (which == 0) mbar_wait_blk(bar, 0);
        else mbar_wait(bar, 0, abort_flag, status);
    }
    __syncthreads();
    if (threadIdx.x == 32) {
        if (which == 0) mbar_wait_blk(bar, 0);
        else mbar_wait(bar, 0, abort_flag, status);
    }
}

}  // namespace

cudaError_t launch_wait_expiry(int which, int32_t* device_status, cudaStream_t st) {
    wait_expiry_kernel<<<1, 64, 0, st>>>(which, device_status);
    return cudaGetLastError();
}

// nibble j = width of step j (bits[j] - bits[j-1]) for lists of at most four widths, else 0
static int i8_wpack(const MoeDims& D) {
    int wpack = 0, prev = 0;
    if (D.K <= 4)
        for (int j = 0; j < D.K; ++j) { wpack |= (D.bits[j] - prev) << (4 * j); prev = D.bits[j]; }
    return wpack;
}

cudaError_t launch_ffn_i8(const d2moe_config* c, const MoeDims& D, const PackLayout& Lgu, const PackLayout& Ld,
                          const ExpertPtrs& P, const __nv_bfloat16* x, const RouteBufs& R, const TcPlan& pl,
                          const TcBuffers& B, int32_t* device_status, cudaStream_t st, void* const* ev,
                          const int32_t* group_keys) {
    auto mark = [&](int i) { if (ev) cudaEventRecord((cudaEvent_t)ev[i], st); };
    const int n_exp = D.E + D.n_shared;
    I8Unit* units = reinterpret_cast<I8Unit*>(B.units);
    float* kappa = B.slot_f;
    float* sigma_x = B.slot_f + pl.R_alloc;
    float* sigma_h = B.slot_f + 2 * pl.R_alloc;
    int8_t* qx = reinterpret_cast<int8_t*>(B.xp16);
    int8_t* qh = reinterpret_cast<int8_t*>(B.h16);
    const int q_blocks = (int)(pl.R_alloc < 1184 ? pl.R_alloc : 1184);

    const int ffn_grid = 2 * device_sm_count();
    size_t prep_smem = (size_t)(D.E * D.K + 1 + n_exp + 1 + pl.max_units + n_exp + 1) * 4;
    if (group_keys) {                       // the grouping's staging area shares the buffer
        const size_t gsm = d2moe_group_is_sortable(D.A, D.E * D.K) ? group_sort_smem_ints(D.A, D.E * D.K, 512 / 32) * 4
                                                                   : (size_t)(((D.A + 31) & ~31) + D.E * D.K + 1) * 4;
        if (gsm > prep_smem) prep_smem = gsm;
    }
    {
        cudaError_t e = ensure_dynamic_smem<&i8_prep_kernel>((int)prep_smem);
        if (e != cudaSuccess) return e;
    }
    // operands of the expert kernels: the width steps themselves when the list has a specialised kernel (the fields of
    // a step are merged in registers), otherwise the stored segments one by one
    const int wp = i8_wpack(D);
    const bool by_step = D.g == 128 && (wp == 0x4112 || wp == 0x422 || wp == 0x1115);
    I8SegMap sm;
    sm.n_seg = by_step ? D.K : Lgu.n_seg;
    for (int j = 0; j < 8; ++j) sm.seg_kk[j] = by_step ? j : Lgu.seg_kk[j];
    launch_chained(i8_prep_kernel, dim3(1), dim3(group_keys ? 512 : 256), prep_smem, st, D, R, units, B.n_units, B.pad_off, B.row_map,
                   B.src_token, kappa, pl.max_units, Lgu.top, Lgu.b1, ffn_grid, device_status, sm, group_keys);
    // threads per slot: a quarter of the row's cells, in whole warps
    auto q_threads = [](int n) { const int t = ((n / 4 + I8_QCPT - 1) / I8_QCPT + 31) & ~31; return t < 1024 ? t : 1024; };
    launch_chained(i8_quant_kernel<true>, dim3(q_blocks), dim3(q_threads(D.d)), 0, st, D.d, D.g, pl.R_alloc, x, B.src_token, B.pad_off, n_exp, kappa,
                                                    qx, B.xk_x, sigma_x, device_status);

    TmaMaps maps_x, maps_h;
    if (!make_maps_u8(&maps_x, qx, 2 * pl.R_alloc, D.d) || !make_maps_u8(&maps_h, qh, 2 * pl.R_alloc, D.F))
        return cudaErrorNotSupported;

    for (int mode = 0; mode < 2; ++mode) {
        I8Params p;
        p.D = D; p.L = mode == 0 ? Lgu : Ld; p.P = P; p.mode = mode;
        p.n_row_tiles = mode == 0 ? D.F / 64 : D.d / 128;
        p.n_split = mode == 0 ? 1 : pl.n_split;
        p.groups_per_split = mode == 0 ? p.L.n_groups : pl.groups_per_split;
        p.units = units; p.n_units = B.n_units; p.next_item = B.n_units + 1 + mode;
        p.xk = mode == 0 ? B.xk_x : B.xk_h;
        p.sigma = mode == 0 ? sigma_x : sigma_h;
        p.hbuf = B.h32; p.obuf = B.o32; p.R_alloc = pl.R_alloc; p.status = device_status;
        const int gps = 128 / D.g;
        const int b_bytes = I8_NSB * I8_B_STAGE;
        const int w_slot = gps * 2 * p.L.block_bytes;
        const int bar_bytes = 512;
        const int budget = 112 * 1024;
        const int rec_bytes = 8 * 40 * 4 + I8_NSQ * 8 * 4;            // per fold warp: the record of its work item; per queue entry: npad
        int nsw = (budget - b_bytes - rec_bytes - 128 - bar_bytes - 1024) / w_slot;
        if (nsw > I8_MAX_NSW) nsw = I8_MAX_NSW;
        if (nsw < 2) return cudaErrorInvalidConfiguration;
        p.nsw = nsw;
        p.smem_w_off = b_bytes;
        p.smem_rec_off = (b_bytes + nsw * w_slot + 127) & ~127;
        p.smem_bar_off = (p.smem_rec_off + rec_bytes + 511) & ~511;   // 512-byte aligned from the 1024-byte aligned base
        const int smem_bytes = p.smem_bar_off + bar_bytes + 1024;
        if (mode == 1)
            launch_chained(i8_quant_kernel<false>, dim3(q_blocks), dim3(q_threads(D.F)), 0, st, D.F, D.g, pl.R_alloc, B.h32,
                           B.src_token, B.pad_off, n_exp, kappa, qh, B.xk_h, sigma_h, device_status);
        mark(mode == 0 ? 1 : 2);
        // width lists of at most four segments that have a specialised kernel (nibble j = width of segment j)
        const int wpack = i8_wpack(D);
        // fold warpgroups: one when a unit is expected to hold few tokens (measured crossover on the Mixtral shape:
        // about 14 tokens per expert), two when the units are full (shared experts take every token)
        const long long per_expert = ((long long)D.A + D.E - 1) / D.E;
        const long long per_unit = D.n_shared > 0 ? (D.T < 32 ? D.T : 32) : 0;
        const int nf = (per_expert <= 12 && per_unit <= 12) ? 1 : 2;
        auto launch = [&](auto kc) -> cudaError_t {
            constexpr auto kern = decltype(kc)::value;
            cudaError_t err = ensure_dynamic_smem<kern>(smem_bytes);
            if (err != cudaSuccess) return err;
            launch_chained(kern, dim3(ffn_grid), dim3(i8_threads(nf)), smem_bytes, st, p, mode == 0 ? maps_x : maps_h);
            return cudaSuccess;
        };
#define I8_KERNEL(GS_, WP_, NF_) std::integral_constant<decltype(&ffn_i8_kernel<GS_, WP_, NF_>), &ffn_i8_kernel<GS_, WP_, NF_>>{}
#define I8_LAUNCH(GS_, WP_) (nf == 1 ? launch(I8_KERNEL(GS_, WP_, 1)) : launch(I8_KERNEL(GS_, WP_, 2)))
        cudaError_t e;
        if (D.g == 128 && wpack == 0x4112) e = I8_LAUNCH(128, 0x4112);        // {2,3,4,8}
        else if (D.g == 128 && wpack == 0x422) e = I8_LAUNCH(128, 0x422);     // {2,4,8}
        else if (D.g == 128 && wpack == 0x1115) e = I8_LAUNCH(128, 0x1115);   // {5,6,7,8}: the 5-bit step stored as 4 + 1
        else if (D.g == 128) e = I8_LAUNCH(128, 0);
        else e = I8_LAUNCH(64, 0);
#undef I8_LAUNCH
#undef I8_KERNEL
        if (e != cudaSuccess) return e;
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}
