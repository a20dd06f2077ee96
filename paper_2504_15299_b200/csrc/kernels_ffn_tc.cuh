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

struct TcPlan {
    int decode;             // 1: memory-bound decode kernel (tokens sorted widest first, one tile per
                            //    segment); 0: grouped dequant-GEMM (one tile per width, any load)
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
};

bool tc_path_supported(const d2moe_config* c);
void tc_plan(const d2moe_config* c, long long T, TcPlan* pl);
cudaError_t launch_ffn_tensor(const d2moe_config* c, const MoeDims& D, const PackLayout& Lgu, const PackLayout& Ld,
                              const ExpertPtrs& P, const __nv_bfloat16* x, const RouteBufs& R, const TcPlan& pl,
                              const TcBuffers& B, int32_t* device_status, cudaStream_t st, void* const* ev);
cudaError_t launch_ffn_decode(const d2moe_config* c, const MoeDims& D, const PackLayout& Lgu, const PackLayout& Ld,
                              const ExpertPtrs& P, const __nv_bfloat16* x, const RouteBufs& R, const TcPlan& pl,
                              const TcBuffers& B, int32_t* device_status, cudaStream_t st, void* const* ev);
