// Shared declarations of the d2moe library: packed-weight layout, workspace carving, launchers.
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/d2moe.h"

#define D2MOE_MAX_SEG 8
#define D2MOE_TILE_ROWS 64          // rows per packed block
#define D2MOE_HEADER_BYTES 256
#define D2MOE_MAGIC 0x4D32444Du     // "MD2M"
#define D2MOE_LAYOUT_VERSION 2u
#define D2MOE_MAX_EXPERTS 320       // routed + shared

// ------------------------------------------------------------------------------------------------
// Programmatic dependent launch for the kernels of one library call.
//
// The kernels of a call form a chain in one stream (route, group, unit build, quantise, expert
// kernels, combine).  Every kernel after the first is launched with the programmatic-serialisation
// attribute: its blocks may be scheduled while the kernel before it is still draining, run their
// set-up, and block in pdl_enter() / pdl_wait() until that kernel has completed and its writes are
// visible.  Every kernel of the chain executes the wait in every block before it reads or writes
// global memory, so completion is transitive along the chain.  The first kernel of a call is an
// ordinary launch.  D2MOE_NO_PDL=1 in the environment turns the attribute off (ordinary launches).
// ------------------------------------------------------------------------------------------------
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_enter() { pdl_wait(); }
#endif

bool d2moe_pdl_enabled();                 // d2moe_api.cu: reads the environment once
inline thread_local bool t_launch_chained = false;
inline void launch_chain_begin() { t_launch_chained = false; }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = (t_launch_chained && d2moe_pdl_enabled()) ? 1 : 0;
    t_launch_chained = true;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// ------------------------------------------------------------------------------------------------
// Packed layout of one [rows, cols] matrix.
//
//   blob   = header (256 B) | block(rt = 0, G = 0) | block(0, 1) | ... | block(n_rt-1, n_groups-1)
//   block  = meta | segment 0 | segment 1 | ...           (64 rows x one group of g input columns)
//   meta   = 64 x (fp16 s1, fp16 lo), row r at byte 4r
//   segment j holds, for each of the 64 rows, the g codes of that segment (bits
//   [shift_j + w_j - 1 : shift_j] of the top-width code) stored sw_j in {1,2,4,8} bits each, i.e.
//   g*sw_j/8 bytes per row, cut in chunks of cs_j = min(16, g*sw_j/8) bytes; chunk c of row r lies
//   at byte (c*64 + r)*cs_j of the segment, so 32 consecutive rows read 32 consecutive chunks.
//   Inside a row's bytes, 32-bit word m holds per = 32/sw codes: the code of element
//   k = m*per + 4*u + i (u < 8/sw, i < 4) sits in byte B(i) = {0, 2, 1, 3}[i] at bit sw*u of that
//   byte.  One AND with a mask that repeats the field at bit sw*u in all four bytes therefore yields
//   the four codes of elements 4u..4u+3 as four 8-bit lanes (byte order k, k+2, k+1, k+3: the operand
//   cell of the 8-bit MMA), and the same AND read as two 16-bit lanes yields the pair (k, k+1) from
//   bytes 0 and 2, and the pair (k+2, k+3) from bytes 1 and 3 after a shift by 8.
//
// A call at width bits[kk] needs meta and segments 0..kk of a block: one contiguous prefix.
//
// Free per-step residual scales (scale_mode 1, Eq. 4 / Eq. 5): segment j >= 1 adds w_j one-bit steps, each
// with its own fp16 scale per (row, group).  Those scales sit directly in front of the segment's codes,
//   block = meta | segment 0 | scales of segment 1 | segment 1 | scales of segment 2 | segment 2 | ...
// as w_j planes of 64 fp16 values (step l of the segment, row r at byte (l*64 + r)*2), so that a call at
// width bits[kk] still reads one contiguous prefix.
// ------------------------------------------------------------------------------------------------
struct PackLayout {
    int rows, cols, g, n_groups, rows_pad, n_rt;
    int n_seg, top, b1;            // n_seg: stored segments (a width step of 3, 5, 6 or 7 bits is stored as 2+1, 4+1, 4+2, 4+2+1)
    int seg_w[D2MOE_MAX_SEG];      // width of stored segment j: 1, 2, 4 or 8 bits
    int seg_sw[D2MOE_MAX_SEG];     // storage width (= seg_w)
    int seg_shift[D2MOE_MAX_SEG];  // position of the segment inside the top-width code
    int seg_cs[D2MOE_MAX_SEG];     // chunk size in bytes
    int seg_off[D2MOE_MAX_SEG + 1];// byte offset of segment j inside a block; [n_seg] = block size
    int seg_kk[D2MOE_MAX_SEG];     // width index whose step the segment belongs to
    int n_widths;                  // number of listed widths
    int last_seg[D2MOE_MAX_SEG];   // width index kk -> its last stored segment (a call at bits[kk] reads segments 0..last_seg[kk])
    int block_bytes;
    int scale_mode;                // 0 tied residual scales, 1 free (one fp16 scale per row, group and extra bit)
    int w_sc_off[D2MOE_MAX_SEG];   // scale_mode 1: byte offset of the scales of width step kk (kk >= 1) inside a block
    int w_lv0[D2MOE_MAX_SEG];      // first residual step (0-based) of width step kk; it has bits[kk] - bits[kk-1] steps
    int w_end[D2MOE_MAX_SEG];      // end of what a call at width index kk reads (bytes from the start of the block)
};

struct PackHeader {
    uint32_t magic, version;
    int32_t rows, cols, g, n_bits;
    int32_t bits[8];
    uint32_t s1_max_bits;          // bit pattern of the largest fp32 s1 in the matrix
    uint32_t wabs_max_bits;        // bit pattern of the largest |W| in the matrix
    int32_t scale_mode;
    uint32_t pad[47];
};
static_assert(sizeof(PackHeader) == D2MOE_HEADER_BYTES, "header size");

__host__ __device__ inline void d2moe_make_layout(PackLayout& L, const int* bits, int n_bits, int g,
                                                  long long rows, long long cols, int scale_mode = 0) {
    L.scale_mode = scale_mode;
    L.rows = (int)rows; L.cols = (int)cols; L.g = g; L.n_groups = (int)(cols / g);
    L.rows_pad = (int)((rows + D2MOE_TILE_ROWS - 1) / D2MOE_TILE_ROWS * D2MOE_TILE_ROWS);
    L.n_rt = L.rows_pad / D2MOE_TILE_ROWS;
    L.top = bits[n_bits - 1]; L.b1 = bits[0]; L.n_widths = n_bits;
    for (int j = 0; j < D2MOE_MAX_SEG; ++j) {
        L.seg_w[j] = L.seg_sw[j] = L.seg_shift[j] = L.seg_cs[j] = L.seg_kk[j] = 0;
        L.last_seg[j] = 0; L.w_sc_off[j] = L.w_lv0[j] = L.w_end[j] = 0;
    }
    int off = D2MOE_TILE_ROWS * 4, prev = 0, n = 0;
    for (int kk = 0; kk < n_bits; ++kk) {
        int w = bits[kk] - prev;                       // the step of this width: stored as power-of-two sub-fields, widest first
        L.w_lv0[kk] = kk == 0 ? 0 : prev - bits[0];
        L.w_sc_off[kk] = off;
        if (scale_mode == 1 && kk >= 1) off += D2MOE_TILE_ROWS * 2 * w;
        int pos = bits[kk] - prev;                     // bits of the step not yet stored
        for (int f = 8; f >= 1; f >>= 1) {
            if (pos >= f && n < D2MOE_MAX_SEG) {
                pos -= f;
                L.seg_w[n] = L.seg_sw[n] = f;
                L.seg_shift[n] = L.top - bits[kk] + pos;
                const int row_bytes = g * f / 8;
                L.seg_cs[n] = row_bytes < 16 ? row_bytes : 16;
                L.seg_off[n] = off;
                L.seg_kk[n] = kk;
                off += D2MOE_TILE_ROWS * row_bytes;
                ++n;
            }
        }
        L.last_seg[kk] = n - 1;
        L.w_end[kk] = off;
        prev = bits[kk];
        (void)w;
    }
    L.n_seg = n;
    for (int j = n; j <= D2MOE_MAX_SEG; ++j) L.seg_off[j] = off;
    L.block_bytes = off;
}

// Byte offset (inside a block) of the 32-bit word that holds element k of row r in segment j, and
// the bit position of the element inside that word.
__host__ __device__ inline int d2moe_elem_word(const PackLayout& L, int j, int r, int k, int* bitpos) {
    int sw = L.seg_sw[j], per = 32 / sw;
    int m = k / per, ko = k - m * per;
    int u = ko >> 2, i = ko & 3;
    int byte = ((i & 1) << 1) | (i >> 1);       // element order inside a cell: bytes 0, 2, 1, 3
    *bitpos = 8 * byte + sw * u;
    int ob = 4 * m, cs = L.seg_cs[j];
    int c = ob / cs, within = ob - c * cs;
    return L.seg_off[j] + (c * D2MOE_TILE_ROWS + r) * cs + within;
}

// scale_mode 1: byte offset (inside a block) of the fp16 scale of residual step `level` (0-based) of row r
__host__ __device__ inline int d2moe_level_offset(const PackLayout& L, int level, int r) {
    int kk = 1;
    while (kk + 1 < L.n_widths && L.w_lv0[kk + 1] <= level) ++kk;
    return L.w_sc_off[kk] + ((level - L.w_lv0[kk]) * D2MOE_TILE_ROWS + r) * 2;
}

// bytes of a block that a call at width index kk reads: meta and the segments (with their scales) of widths 0..kk
__host__ __device__ inline int d2moe_prefix_bytes(const PackLayout& L, int kk) { return L.w_end[kk]; }

__host__ __device__ inline size_t d2moe_block_offset(const PackLayout& L, int rt, int G) {
    return (size_t)D2MOE_HEADER_BYTES + ((size_t)rt * L.n_groups + G) * (size_t)L.block_bytes;
}

// ------------------------------------------------------------------------------------------------
// Problem description handed to the kernels (by value).
// ------------------------------------------------------------------------------------------------
struct MoeDims {
    int T, d, F, E, k, n_shared, g, K;   // K = n_bits
    int bits[8];
    int A;        // routed assignments T*k
    int A_tot;    // A + n_shared*T
    int renormalize;
};

struct ExpertPtrs {                       // [expert][gate, up, down]
    const uint8_t* w[3 * D2MOE_MAX_EXPERTS];
};

struct RouteBufs {
    int32_t* topk_idx; float* topk_w; int8_t* bit_idx;
    int32_t* perm; int32_t* inv_perm; int32_t* group_off;
};

// Grouping of the assignments by (expert, width) key: the single-block kernel takes the smallest loads (its
// rule is in launch_route), a single-block counting sort loads of up to 4096 assignments on up to 512 keys, one
// launch of a few blocks the other mid-sized ones (every block counts all keys: the walks per warp must stay
// short), histogram + scan + scatter kernels the rest.  All give the same (unique) stable order.
static inline bool d2moe_group_is_mid(long long A, long long n_keys) {
    return A <= 12288 && n_keys <= 2048 && n_keys * ((A + 31) / 32) <= 6144;
}

// Workspace carving (all offsets 256-byte aligned).
struct Workspace {
    size_t total;
    size_t off_logits, off_keys, off_hist;
    size_t off_topk_idx, off_topk_w, off_bit_idx, off_perm, off_inv_perm, off_group_off;
    size_t off_h, off_o, off_status;
    size_t off_units, off_n_units, off_pad_off, off_row_map, off_src_token, off_xp16;   // tensor-core path
    size_t off_h32, off_xk_x, off_xk_h, off_slot_f;                                     // 8-bit decode kernel
};

void d2moe_carve_workspace(const d2moe_config* cfg, long long max_tokens, Workspace* ws);

// kernels_pack.cu
cudaError_t launch_pack(const PackLayout& L, const int* bits, int n_bits, const float* W, uint8_t* packed,
                        cudaStream_t st);
cudaError_t launch_pack_calibrated(const PackLayout& L, const int* bits, int n_bits, float* W, const float* hc,
                                   const float* col_energy, uint8_t* packed, cudaStream_t st);
cudaError_t launch_unpack(const PackLayout& L, const uint8_t* packed, int bits, uint8_t* codes,
                          float* scale, float* offset, cudaStream_t st);
cudaError_t launch_unpack_scales(const PackLayout& L, const uint8_t* packed, float* s_extra, cudaStream_t st);

// kernels_route.cu
cudaError_t launch_route(const MoeDims& D, const __nv_bfloat16* x, const __nv_bfloat16* gate_w,
                         const float* logits_in, const __nv_bfloat16* bit_w, const int8_t* forced,
                         const RouteBufs& R, float* logits_ws, int32_t* keys_ws, int32_t* hist_ws,
                         int32_t* device_status, cudaStream_t st, bool* defer_small_group = nullptr);
// the single-block grouping rule of launch_route (decode-sized loads)
static inline bool d2moe_group_is_small(long long A, long long n_keys) {
    return A <= 8192 && n_keys <= 2048 && n_keys * ((A + 31) / 32) <= 1024;
}
// loads that one block groups by a counting sort (in front of the decode path's unit build)
#ifdef __CUDACC__
__host__ __device__
#endif
static inline bool d2moe_group_is_sortable(long long A, long long n_keys) { return A <= 4096 && n_keys <= 512; }

// kernels_ffn_cc.cu  (plain CUDA-core path)
cudaError_t launch_gateup_cuda_core(const MoeDims& D, const PackLayout& Lgu, const ExpertPtrs& P,
                                    const __nv_bfloat16* x, const RouteBufs& R, float* hbuf,
                                    int32_t* device_status, cudaStream_t st);
cudaError_t launch_down_cuda_core(const MoeDims& D, const PackLayout& Ld, const ExpertPtrs& P,
                                  const RouteBufs& R, const float* hbuf, float* obuf,
                                  int32_t* device_status, cudaStream_t st);
cudaError_t launch_combine(const MoeDims& D, const RouteBufs& R, const float* obuf, int n_split,
                           size_t split_stride, const int32_t* row_map, const __nv_bfloat16* residual,
                           __nv_bfloat16* y, cudaStream_t st);
cudaError_t launch_rmsnorm(int T, int d, float eps, const __nv_bfloat16* x, __nv_bfloat16* xn, cudaStream_t st);
