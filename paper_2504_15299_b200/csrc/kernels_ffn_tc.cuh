// Interface of the tensor-core (tcgen05) expert path.
#pragma once
#include "d2moe_common.cuh"

// Up to n_cap consecutive padded rows (tokens) of one expert: one piece per routed width.
struct TcUnit {
    int e;         // expert (routed, then shared)
    int row0;      // first padded row in the gathered activation buffers
    int ncols;     // rows in this unit (multiple of 16, <= n_cap)
    int kmax;      // highest width index present
    int col0[8];   // first column of the piece of width index kk inside the unit
    int cnt[8];    // its padded columns inside the unit (multiple of 16, 0 = absent)
    int real[8];   // its real (non-padding) columns inside the unit
};

// Unit of the 8-bit decode kernel: up to 32 consecutive token slots of one expert.  The slots of an
// expert are laid out by width, widest first, every width class padded to a multiple of 8 slots, so
// the slots that include segment j are the first npad[j] slots of the unit.
struct I8Unit {
    int e;         // expert (routed, then shared)
    int slot0;     // first slot (multiple of 8); the quantised activations of slot s are rows 2s, 2s+1
    int nslots;    // slots in this unit (multiple of 8, <= 32)
    int kmax;      // last stored segment any of its tokens reads
    int nblk;      // blocks of 4 slots that hold at least one real token
    int npad[8];   // slots covered by the product of stored segment j (multiple of 8, 0 = absent)
    int blk[8];    // the real blocks: first slot / 4, relative to slot0
};

// largest average number of tokens per expert that the 8-bit decode kernel takes
#define D2MOE_DECODE_MAX_AVG 40

struct TcPlan {
    int decode;             // 1: memory-bound 8-bit decode kernel (tokens laid out widest first, scales applied
                            //    to the accumulators); 0: grouped fp16 dequant-GEMM (one tile per width, any load)
    int n_cap;              // columns per unit
    long long R_alloc;      // rows of the padded activation buffers
    int max_units;
    int n_split, groups_per_split;   // split-K of the down projection
};

struct TcBuffers {
    TcUnit* units; int* n_units; int32_t* pad_off; int32_t* row_map; int32_t* src_token;
    __half* xp16;           // [R_alloc, d]   gathered tokens, fp16
    __half* h16;            // [R_alloc, F]   SwiGLU outputs, fp16
    float* o32;             // [n_split][R_alloc, d] partial expert outputs
    // 8-bit decode kernel: xp16 / h16 are reused as the quantised activations [2 R_alloc, d] / [2 R_alloc, F]
    float* h32;             // [R_alloc, F]   SwiGLU outputs, fp32
    float* xk_x;            // [d / g][R_alloc][2]   per group and slot: sum of the quantised x, kappa * sum
    float* xk_h;            // [F / g][R_alloc][2]
    float* slot_f;          // [3][R_alloc]   decode kernel: kappa, scale of x, scale of h per slot; grouped GEMM: the three
                            //                power-of-two factors of the per-row activation scaling
};

bool tc_path_supported(const d2moe_config* c);
cudaError_t launch_wait_expiry(int which, int32_t* device_status, cudaStream_t st);
void tc_plan(const d2moe_config* c, long long T, TcPlan* pl);
cudaError_t launch_ffn_tensor(const d2moe_config* c, const MoeDims& D, const PackLayout& Lgu, const PackLayout& Ld,
                              const ExpertPtrs& P, const __nv_bfloat16* x, const RouteBufs& R, const TcPlan& pl,
                              const TcBuffers& B, int32_t* device_status, cudaStream_t st, void* const* ev);
// group_keys: when not null, the sort keys of the assignments whose grouping (group_off, perm, inv_perm of R) is
// still to be done: the unit build does it first, in the same launch
cudaError_t launch_ffn_i8(const d2moe_config* c, const MoeDims& D, const PackLayout& Lgu, const PackLayout& Ld,
                          const ExpertPtrs& P, const __nv_bfloat16* x, const RouteBufs& R, const TcPlan& pl,
                          const TcBuffers& B, int32_t* device_status, cudaStream_t st, void* const* ev,
                          const int32_t* group_keys = nullptr);
