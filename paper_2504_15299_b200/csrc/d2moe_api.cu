// Host side of the C ABI: argument checks, workspace carving, launches.
#include "d2moe_common.cuh"
#include <cstdlib>
#include "kernels_ffn_tc.cuh"

#include <string.h>

bool d2moe_pdl_enabled() {
    static const bool on = [] { const char* e = getenv("D2MOE_NO_PDL"); return !(e && e[0] == '1'); }();
    return on;
}

namespace {

inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

bool fill_dims(const d2moe_config* c, long long T, MoeDims* D) {
    D->T = (int)T; D->d = c->d_model; D->F = c->d_ffn; D->E = c->n_experts; D->k = c->top_k;
    D->n_shared = c->n_shared; D->g = c->group_size; D->K = c->n_bits;
    for (int i = 0; i < 8; ++i) D->bits[i] = i < c->n_bits ? c->bits[i] : 0;
    D->A = (int)(T * c->top_k);
    D->A_tot = D->A + (int)(T * c->n_shared);
    D->renormalize = c->renormalize;
    return true;
}

}  // namespace

extern "C" const char* d2moe_status_string(d2moe_status s) {
    switch (s) {
        case D2MOE_OK: return "ok";
        case D2MOE_ERR_NULL: return "a required pointer is NULL";
        case D2MOE_ERR_CONFIG: return "inconsistent configuration";
        case D2MOE_ERR_SHAPE: return "size does not fit the configuration";
        case D2MOE_ERR_UNSUPPORTED: return "valid but not supported by this build";
        case D2MOE_ERR_WORKSPACE: return "workspace or output buffer too small";
        case D2MOE_ERR_CUDA: return "CUDA call or launch failed";
        case D2MOE_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case D2MOE_ERR_NONFINITE: return "non-finite router logit";
    }
    return "unknown status";
}

extern "C" d2moe_status d2moe_check_config(const d2moe_config* c) {
    if (!c) return D2MOE_ERR_NULL;
    if (c->d_model <= 0 || c->d_ffn <= 0 || c->n_experts <= 0 || c->top_k <= 0 || c->n_shared < 0)
        return D2MOE_ERR_CONFIG;
    if (c->top_k > c->n_experts || c->top_k > 8) return D2MOE_ERR_CONFIG;
    if (c->d_model > D2MOE_MAX_DIM || c->d_ffn > D2MOE_MAX_DIM) return D2MOE_ERR_CONFIG;   // what every launch can take
    if (c->n_experts > 256 || c->n_experts + c->n_shared > D2MOE_MAX_EXPERTS) return D2MOE_ERR_CONFIG;
    const int g = c->group_size;
    if (!(g == 32 || g == 64 || g == 128 || g == 256)) return D2MOE_ERR_CONFIG;
    if (c->d_model % g || c->d_ffn % g) return D2MOE_ERR_CONFIG;
    if (c->n_bits < 1 || c->n_bits > 8) return D2MOE_ERR_CONFIG;
    if (c->bits[0] < 1 || c->bits[c->n_bits - 1] > 8) return D2MOE_ERR_CONFIG;
    for (int i = 1; i < c->n_bits; ++i)
        if (c->bits[i] <= c->bits[i - 1]) return D2MOE_ERR_CONFIG;
    if (c->renormalize != 0 && c->renormalize != 1) return D2MOE_ERR_CONFIG;
    if (c->scale_mode != 0 && c->scale_mode != 1) return D2MOE_ERR_CONFIG;
    if (c->kernel_path < 0 || c->kernel_path > 2) return D2MOE_ERR_CONFIG;
    for (int i = 0; i < 3; ++i)
        if (c->reserved[i] != 0) return D2MOE_ERR_CONFIG;
    return D2MOE_OK;
}

extern "C" d2moe_status d2moe_packed_bytes(const d2moe_config* c, int64_t rows, int64_t cols,
                                           size_t* total_bytes, size_t* code_bytes, size_t* meta_bytes) {
    d2moe_status s = d2moe_check_config(c);
    if (s != D2MOE_OK) return s;
    if (!total_bytes) return D2MOE_ERR_NULL;
    if (rows <= 0 || cols <= 0 || cols % c->group_size || rows > (1 << 24) || cols > (1 << 24))
        return D2MOE_ERR_SHAPE;
    PackLayout L;
    d2moe_make_layout(L, c->bits, c->n_bits, c->group_size, rows, cols, c->scale_mode);
    const size_t n_blocks = (size_t)L.n_rt * L.n_groups;
    const size_t n_steps = c->scale_mode == 1 ? (size_t)(L.top - L.b1) : 0;       // free scales: one fp16 per extra bit
    const size_t meta = n_blocks * D2MOE_TILE_ROWS * (4 + 2 * n_steps);
    const size_t code = n_blocks * (size_t)L.block_bytes - meta;
    *total_bytes = D2MOE_HEADER_BYTES + meta + code;
    if (code_bytes) *code_bytes = code;
    if (meta_bytes) *meta_bytes = meta;
    return D2MOE_OK;
}

extern "C" d2moe_status d2moe_pack_mwq(const d2moe_config* c, const float* W, int64_t rows, int64_t cols,
                                       void* packed, size_t packed_bytes, void* stream) {
    size_t need = 0;
    d2moe_status s = d2moe_packed_bytes(c, rows, cols, &need, nullptr, nullptr);
    if (s != D2MOE_OK) return s;
    if (!W || !packed) return D2MOE_ERR_NULL;
    if (packed_bytes < need) return D2MOE_ERR_WORKSPACE;
    if (((uintptr_t)packed & 255) != 0) return D2MOE_ERR_SHAPE;
    PackLayout L;
    d2moe_make_layout(L, c->bits, c->n_bits, c->group_size, rows, cols, c->scale_mode);
    cudaError_t e = launch_pack(L, c->bits, c->n_bits, W, (uint8_t*)packed, (cudaStream_t)stream);
    return e == cudaSuccess ? D2MOE_OK : D2MOE_ERR_CUDA;
}

extern "C" d2moe_status d2moe_pack_mwq_calibrated(const d2moe_config* c, float* W, int64_t rows, int64_t cols,
                                                  const float* hc, const float* col_energy, void* packed,
                                                  size_t packed_bytes, void* stream) {
    size_t need = 0;
    d2moe_status s = d2moe_packed_bytes(c, rows, cols, &need, nullptr, nullptr);
    if (s != D2MOE_OK) return s;
    if (c->scale_mode != 1) return D2MOE_ERR_CONFIG;         // the scale fit of Eq. 5 needs the free scales
    if (!W || !packed) return D2MOE_ERR_NULL;
    if (packed_bytes < need) return D2MOE_ERR_WORKSPACE;
    if (((uintptr_t)packed & 255) != 0) return D2MOE_ERR_SHAPE;
    PackLayout L;
    d2moe_make_layout(L, c->bits, c->n_bits, c->group_size, rows, cols, c->scale_mode);
    cudaError_t e = launch_pack_calibrated(L, c->bits, c->n_bits, W, hc, col_energy, (uint8_t*)packed, (cudaStream_t)stream);
    return e == cudaSuccess ? D2MOE_OK : D2MOE_ERR_CUDA;
}

extern "C" d2moe_status d2moe_unpack_codes(const d2moe_config* c, const void* packed, int64_t rows,
                                           int64_t cols, int bits, uint8_t* codes, float* scale,
                                           float* offset, void* stream) {
    size_t need = 0;
    d2moe_status s = d2moe_packed_bytes(c, rows, cols, &need, nullptr, nullptr);
    if (s != D2MOE_OK) return s;
    if (!packed || !codes) return D2MOE_ERR_NULL;
    if (bits < c->bits[0] || bits > c->bits[c->n_bits - 1]) return D2MOE_ERR_SHAPE;
    PackLayout L;
    d2moe_make_layout(L, c->bits, c->n_bits, c->group_size, rows, cols, c->scale_mode);
    cudaError_t e = launch_unpack(L, (const uint8_t*)packed, bits, codes, scale, offset, (cudaStream_t)stream);
    return e == cudaSuccess ? D2MOE_OK : D2MOE_ERR_CUDA;
}

extern "C" d2moe_status d2moe_unpack_scales(const d2moe_config* c, const void* packed, int64_t rows,
                                            int64_t cols, float* s_extra, void* stream) {
    size_t need = 0;
    d2moe_status s = d2moe_packed_bytes(c, rows, cols, &need, nullptr, nullptr);
    if (s != D2MOE_OK) return s;
    if (c->scale_mode != 1) return D2MOE_ERR_CONFIG;
    if (!packed || !s_extra) return D2MOE_ERR_NULL;
    PackLayout L;
    d2moe_make_layout(L, c->bits, c->n_bits, c->group_size, rows, cols, c->scale_mode);
    cudaError_t e = launch_unpack_scales(L, (const uint8_t*)packed, s_extra, (cudaStream_t)stream);
    return e == cudaSuccess ? D2MOE_OK : D2MOE_ERR_CUDA;
}

// AUTO takes the tensor-core path whenever the shape allows it; TENSOR insists on it.
static bool use_tensor_path(const d2moe_config* c) {
    return c->kernel_path != D2MOE_PATH_CUDA_CORE && tc_path_supported(c);
}

void d2moe_carve_workspace(const d2moe_config* c, long long T, Workspace* ws) {
    const size_t A = (size_t)T * c->top_k;
    const size_t A_tot = A + (size_t)T * c->n_shared;
    const size_t n_keys = (size_t)c->n_experts * c->n_bits;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align256(off + bytes); return o; };
    ws->off_status = take(256);
    ws->off_logits = take((size_t)T * c->n_experts * 4);
    ws->off_keys = take(A * 4);
    ws->off_hist = take(n_keys * 4);
    ws->off_topk_idx = take(A * 4);
    ws->off_topk_w = take(A * 4);
    ws->off_bit_idx = take(A);
    ws->off_perm = take(A * 4);
    ws->off_inv_perm = take(A * 4);
    ws->off_group_off = take((n_keys + 1) * 4);
    if (use_tensor_path(c)) {
        TcPlan pl;
        tc_plan(c, T, &pl);
        ws->off_units = take((size_t)pl.max_units * sizeof(TcUnit));
        ws->off_n_units = take(256);
        ws->off_pad_off = take((n_keys + c->n_shared + 1) * 4);
        ws->off_row_map = take(A_tot * 4);
        ws->off_src_token = take((size_t)pl.R_alloc * 4);
        ws->off_xp16 = take((size_t)pl.R_alloc * c->d_model * 2);
        ws->off_h = take((size_t)pl.R_alloc * c->d_ffn * 2);
        // the split-K factor of the down projection falls as the batch grows: size the partial outputs for
        // the smallest batch that takes the same kernel, so that the total never shrinks when T grows
        TcPlan pl_lo;
        const long long t_dec = (long long)D2MOE_DECODE_MAX_AVG * c->n_experts / c->top_k;
        tc_plan(c, pl.decode ? 1 : (t_dec + 1 < T ? t_dec + 1 : T), &pl_lo);
        const int n_split_alloc = pl_lo.n_split > pl.n_split ? pl_lo.n_split : pl.n_split;
        ws->off_o = take((size_t)n_split_alloc * pl.R_alloc * c->d_model * 4);
        ws->off_h32 = ws->off_xk_x = ws->off_xk_h = 0;
        ws->off_slot_f = take((size_t)3 * pl.R_alloc * 4);      // per padded row: three scale factors (either kernel)
        if (pl.decode) {
            ws->off_h32 = take((size_t)pl.R_alloc * c->d_ffn * 4);
            ws->off_xk_x = take((size_t)(c->d_model / c->group_size) * pl.R_alloc * 8);
            ws->off_xk_h = take((size_t)(c->d_ffn / c->group_size) * pl.R_alloc * 8);
        }
    } else {
        ws->off_units = ws->off_n_units = ws->off_pad_off = ws->off_row_map = ws->off_src_token = ws->off_xp16 = 0;
        ws->off_h32 = ws->off_xk_x = ws->off_xk_h = ws->off_slot_f = 0;
        ws->off_h = take(A_tot * (size_t)c->d_ffn * 4);
        ws->off_o = take(A_tot * (size_t)c->d_model * 4);
    }
    ws->total = off;
}

extern "C" size_t d2moe_workspace_bytes(const d2moe_config* c, int64_t max_tokens) {
    if (d2moe_check_config(c) != D2MOE_OK || max_tokens < 0 || max_tokens > (1 << 20)) return 0;
    const long long T = max_tokens > 0 ? max_tokens : 1;
    Workspace ws;
    d2moe_carve_workspace(c, T, &ws);
    size_t total = ws.total;
    // a call with fewer tokens may take the other expert kernel, whose buffers are laid out differently:
    // cover the largest batch of that kind as well, so that every T <= max_tokens fits
    const long long t_dec = (long long)D2MOE_DECODE_MAX_AVG * c->n_experts / c->top_k;      // largest batch the decode kernel takes
    if (t_dec >= 1 && t_dec < T) {
        d2moe_carve_workspace(c, t_dec, &ws);
        if (ws.total > total) total = ws.total;
    }
    return total;
}

static d2moe_status check_route_inputs(const void* gate_w, const float* logits, const void* bit_w,
                                       const int8_t* forced) {
    if ((gate_w == nullptr) == (logits == nullptr)) return D2MOE_ERR_NULL;
    if ((bit_w == nullptr) == (forced == nullptr)) return D2MOE_ERR_NULL;
    return D2MOE_OK;
}

extern "C" d2moe_status d2moe_route(const d2moe_config* c, int64_t T, const void* x, const void* gate_w,
                                    const float* logits, const void* bit_w, const int8_t* forced,
                                    int32_t* topk_idx, float* topk_w, int8_t* bit_idx, int32_t* perm,
                                    int32_t* inv_perm, int32_t* group_off, int32_t* device_status,
                                    void* workspace, size_t workspace_bytes, void* stream) {
    d2moe_status s = d2moe_check_config(c);
    if (s != D2MOE_OK) return s;
    if (T < 0 || T > (1 << 20)) return D2MOE_ERR_SHAPE;
    if (!topk_idx || !topk_w || !bit_idx || !perm || !inv_perm || !group_off) return D2MOE_ERR_NULL;
    if (T > 0 && !x) return D2MOE_ERR_NULL;
    s = check_route_inputs(gate_w, logits, bit_w, forced);
    if (s != D2MOE_OK) return s;
    if (!workspace) return D2MOE_ERR_NULL;
    Workspace ws;
    d2moe_carve_workspace(c, T > 0 ? T : 1, &ws);
    if (workspace_bytes < ws.total) return D2MOE_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    MoeDims D;
    fill_dims(c, T, &D);
    const int n_keys = D.E * D.K;
    if (T == 0) {
        cudaError_t e = cudaMemsetAsync(group_off, 0, (size_t)(n_keys + 1) * 4, st);
        return e == cudaSuccess ? D2MOE_OK : D2MOE_ERR_CUDA;
    }
    uint8_t* w = (uint8_t*)workspace;
    RouteBufs R{topk_idx, topk_w, bit_idx, perm, inv_perm, group_off};
    launch_chain_begin();
    cudaError_t e = launch_route(D, (const __nv_bfloat16*)x, (const __nv_bfloat16*)gate_w, logits,
                                 (const __nv_bfloat16*)bit_w, forced, R, (float*)(w + ws.off_logits),
                                 (int32_t*)(w + ws.off_keys), (int32_t*)(w + ws.off_hist), device_status, st);
    return e == cudaSuccess ? D2MOE_OK : D2MOE_ERR_CUDA;
}

// Host-side checks of a forward call; nothing is launched before they pass.
static d2moe_status validate_forward(const d2moe_config* c, int64_t T, const void* x,
                                     const void* const* expert_w, const d2moe_route_in* in,
                                     const d2moe_route_out* pre, const void* y, const void* workspace,
                                     size_t workspace_bytes) {
    d2moe_status s = d2moe_check_config(c);
    if (s != D2MOE_OK) return s;
    if (T < 0 || T > (1 << 20)) return D2MOE_ERR_SHAPE;
    if (T == 0) return D2MOE_OK;
    if (!x || !expert_w || !y || !workspace) return D2MOE_ERR_NULL;
    if (!pre && !in) return D2MOE_ERR_NULL;
    const int n_exp = c->n_experts + c->n_shared;
    for (int i = 0; i < 3 * n_exp; ++i)
        if (!expert_w[i]) return D2MOE_ERR_NULL;
    if (pre) {
        if (!pre->topk_idx || !pre->topk_w || !pre->bit_idx || !pre->perm || !pre->inv_perm || !pre->group_off)
            return D2MOE_ERR_NULL;
    } else {
        s = check_route_inputs(in->gate_w_bf16, in->logits, in->bit_w_bf16, in->forced_bit_idx);
        if (s != D2MOE_OK) return s;
    }
    if (c->kernel_path == D2MOE_PATH_TENSOR && !tc_path_supported(c)) return D2MOE_ERR_UNSUPPORTED;
    Workspace ws;
    d2moe_carve_workspace(c, T, &ws);
    if (workspace_bytes < ws.total) return D2MOE_ERR_WORKSPACE;
    return D2MOE_OK;
}

static d2moe_status forward_impl(const d2moe_config* c, int64_t T, const void* x, const void* const* expert_w,
                                 const d2moe_route_in* in, const d2moe_route_out* pre,
                                 const void* residual, void* y, int32_t* device_status, void* workspace,
                                 size_t workspace_bytes, cudaStream_t st, void* const* ev = nullptr,
                                 bool continue_chain = false) {
    d2moe_status s = validate_forward(c, T, x, expert_w, in, pre, y, workspace, workspace_bytes);
    if (s != D2MOE_OK || T == 0) return s;
    if (!continue_chain) launch_chain_begin();
    const int n_exp = c->n_experts + c->n_shared;
    Workspace ws;
    d2moe_carve_workspace(c, T, &ws);

    MoeDims D;
    fill_dims(c, T, &D);
    uint8_t* w = (uint8_t*)workspace;
    RouteBufs R;
    cudaError_t e;
    auto mark = [&](int i) { if (ev) cudaEventRecord((cudaEvent_t)ev[i], st); };
    mark(0);
    bool want_defer = false, group_deferred = false;
    if (pre) {
        R = RouteBufs{(int32_t*)pre->topk_idx, (float*)pre->topk_w, (int8_t*)pre->bit_idx,
                      (int32_t*)pre->perm, (int32_t*)pre->inv_perm, (int32_t*)pre->group_off};
    } else {
        R = RouteBufs{(int32_t*)(w + ws.off_topk_idx), (float*)(w + ws.off_topk_w), (int8_t*)(w + ws.off_bit_idx),
                      (int32_t*)(w + ws.off_perm), (int32_t*)(w + ws.off_inv_perm),
                      (int32_t*)(w + ws.off_group_off)};
        // decode-sized loads on the 8-bit kernel: the grouping runs in front of that path's unit build, in one launch
        if (use_tensor_path(c)) {
            TcPlan pl0;
            tc_plan(c, T, &pl0);
            want_defer = pl0.decode != 0;
        }
        e = launch_route(D, (const __nv_bfloat16*)x, (const __nv_bfloat16*)in->gate_w_bf16, in->logits,
                         (const __nv_bfloat16*)in->bit_w_bf16, in->forced_bit_idx, R,
                         (float*)(w + ws.off_logits), (int32_t*)(w + ws.off_keys),
                         (int32_t*)(w + ws.off_hist), device_status, st, want_defer ? &group_deferred : nullptr);
        if (e != cudaSuccess) return D2MOE_ERR_CUDA;
    }
    ExpertPtrs P;
    memset(&P, 0, sizeof(P));
    for (int i = 0; i < 3 * n_exp; ++i) P.w[i] = (const uint8_t*)expert_w[i];
    PackLayout Lgu, Ld;
    d2moe_make_layout(Lgu, c->bits, c->n_bits, c->group_size, c->d_ffn, c->d_model, c->scale_mode);
    d2moe_make_layout(Ld, c->bits, c->n_bits, c->group_size, c->d_model, c->d_ffn, c->scale_mode);

    if (use_tensor_path(c)) {
        TcPlan pl;
        tc_plan(c, T, &pl);
        TcBuffers B;
        B.units = (TcUnit*)(w + ws.off_units); B.n_units = (int*)(w + ws.off_n_units);
        B.pad_off = (int32_t*)(w + ws.off_pad_off); B.row_map = (int32_t*)(w + ws.off_row_map);
        B.src_token = (int32_t*)(w + ws.off_src_token);
        B.xp16 = (__half*)(w + ws.off_xp16); B.h16 = (__half*)(w + ws.off_h); B.o32 = (float*)(w + ws.off_o);
        B.h32 = (float*)(w + ws.off_h32); B.xk_x = (float*)(w + ws.off_xk_x); B.xk_h = (float*)(w + ws.off_xk_h);
        B.slot_f = (float*)(w + ws.off_slot_f);
        e = pl.decode ? launch_ffn_i8(c, D, Lgu, Ld, P, (const __nv_bfloat16*)x, R, pl, B, device_status, st, ev,
                                      group_deferred ? (const int32_t*)(w + ws.off_keys) : nullptr)
                      : launch_ffn_tensor(c, D, Lgu, Ld, P, (const __nv_bfloat16*)x, R, pl, B, device_status, st, ev);
        if (e != cudaSuccess) return D2MOE_ERR_CUDA;
        mark(3);
        e = launch_combine(D, R, B.o32, pl.n_split, (size_t)pl.R_alloc * D.d, B.row_map,
                           (const __nv_bfloat16*)residual, (__nv_bfloat16*)y, st);
        mark(4);
        return e == cudaSuccess ? D2MOE_OK : D2MOE_ERR_CUDA;
    }
    float* hbuf = (float*)(w + ws.off_h);
    float* obuf = (float*)(w + ws.off_o);
    mark(1);
    e = launch_gateup_cuda_core(D, Lgu, P, (const __nv_bfloat16*)x, R, hbuf, device_status, st);
    if (e != cudaSuccess) return D2MOE_ERR_CUDA;
    mark(2);
    e = launch_down_cuda_core(D, Ld, P, R, hbuf, obuf, device_status, st);
    if (e != cudaSuccess) return D2MOE_ERR_CUDA;
    mark(3);
    e = launch_combine(D, R, obuf, 1, (size_t)D.A_tot * D.d, nullptr, (const __nv_bfloat16*)residual,
                       (__nv_bfloat16*)y, st);
    mark(4);
    return e == cudaSuccess ? D2MOE_OK : D2MOE_ERR_CUDA;
}

extern "C" d2moe_status d2moe_moe_forward(const d2moe_config* c, int64_t T, const void* x,
                                          const void* const* expert_w, const d2moe_route_in* in,
                                          const d2moe_route_out* pre, void* y, int32_t* device_status,
                                          void* workspace, size_t workspace_bytes, void* stream) {
    return forward_impl(c, T, x, expert_w, in, pre, nullptr, y, device_status, workspace, workspace_bytes,
                        (cudaStream_t)stream);
}

extern "C" d2moe_status d2moe_moe_forward_events(const d2moe_config* c, int64_t T, const void* x,
                                                 const void* const* expert_w, const d2moe_route_in* in,
                                                 const d2moe_route_out* pre, void* y, int32_t* device_status,
                                                 void* workspace, size_t workspace_bytes, void* stream,
                                                 void* const* stage_events) {
    if (!stage_events) return D2MOE_ERR_NULL;
    for (int i = 0; i <= D2MOE_N_STAGES; ++i)
        if (!stage_events[i]) return D2MOE_ERR_NULL;
    return forward_impl(c, T, x, expert_w, in, pre, nullptr, y, device_status, workspace, workspace_bytes,
                        (cudaStream_t)stream, stage_events);
}

extern "C" d2moe_status d2moe_selftest_wait_expiry(int which, int32_t* device_status, void* stream) {
    if (!device_status) return D2MOE_ERR_NULL;
    if (which < 0 || which > 1) return D2MOE_ERR_SHAPE;
    return launch_wait_expiry(which, device_status, (cudaStream_t)stream) == cudaSuccess ? D2MOE_OK : D2MOE_ERR_CUDA;
}

extern "C" int d2moe_forward_launch_count(const d2moe_config* c, int64_t T, int routing_precomputed) {
    if (d2moe_check_config(c) != D2MOE_OK || T <= 0) return 0;
    // route, then count + scan + scatter (one launch when the load is small: the rule of launch_route)
    const long long A = (long long)T * c->top_k, n_keys = (long long)c->n_experts * c->n_bits;
    const bool small = A <= 8192 && n_keys <= 2048 && n_keys * ((A + 31) / 32) <= 1024;
    int route = routing_precomputed ? 0 : (small || d2moe_group_is_sortable(A, n_keys) || d2moe_group_is_mid(A, n_keys) ? 2 : 4);
    if (!routing_precomputed && (small || d2moe_group_is_sortable(A, n_keys)) && use_tensor_path(c)) {   // grouping inside the decode path's unit build
        TcPlan pl0;
        tc_plan(c, T, &pl0);
        if (pl0.decode) route -= 1;
    }
    // more than 16 experts: the gate logits come from a tiled kernel of their own (when the caller supplies
    // logits instead of gate weights that launch does not happen: the count is then one too high)
    if (!routing_precomputed && c->n_experts > 16 && (size_t)c->d_model * 2 * 16 <= 200 * 1024) route += 1;
    if (use_tensor_path(c)) {
        TcPlan pl;
        tc_plan(c, T, &pl);
        // unit build, gather (decode: quantise x), gate/up, (decode: quantise h), down, combine
        return route + (pl.decode ? 6 : 5);
    }
    return route + 3;                                   // gate/up, down, combine
}

extern "C" d2moe_status d2moe_stack_layer(const d2moe_config* c, int64_t T, void* x, void* xn, float eps,
                                          const void* const* expert_w, const d2moe_route_in* in,
                                          int32_t* device_status, void* workspace, size_t workspace_bytes,
                                          void* stream) {
    if (T > 0 && (!x || !xn || !in)) return D2MOE_ERR_NULL;
    d2moe_status s = validate_forward(c, T, xn, expert_w, in, nullptr, x, workspace, workspace_bytes);
    if (s != D2MOE_OK || T == 0) return s;
    if (!(eps >= 0.0f)) return D2MOE_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    launch_chain_begin();
    cudaError_t e = launch_rmsnorm((int)T, c->d_model, eps, (const __nv_bfloat16*)x, (__nv_bfloat16*)xn, st);
    if (e != cudaSuccess) return D2MOE_ERR_CUDA;
    return forward_impl(c, T, xn, expert_w, in, nullptr, x, x, device_status, workspace, workspace_bytes, st, nullptr, true);
}
