/*
 * d2moe.h - C ABI of the B200 (sm_100a) dual-routed MoE layer over matryoshka-weight-quantized
 * (MWQ) experts, after "D2MoE: Dual Routing and Dynamic Scheduling for Efficient On-Device
 * MoE-based LLM Serving" (Sections 3.2 and 3.3).
 *
 * Conventions for every entry point
 *   - "device" pointers are CUDA device memory of the current device, "host" pointers are host
 *     memory.  The caller owns every buffer; the library allocates nothing and keeps no state
 *     between calls (unless an entry point's comment says otherwise).
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = default stream) and the
 *     call returns without synchronising.  The kernels of one call are launched as programmatic
 *     dependents of one another (each waits on the device for the one before it; the first kernel
 *     of a call is an ordinary launch); the environment variable D2MOE_NO_PDL=1, read once, makes
 *     every launch an ordinary one.
 *   - The return value reports what the host can see before and at launch: null pointers, bad
 *     configuration or shapes, short buffers, a failed launch.  Nothing is launched when an
 *     argument check fails.  Anomalies only the device can see (non-finite router logits, a bounded
 *     wait that ran out) are OR-ed into the optional `device_status` word, which the caller reads
 *     after its own synchronisation.  No call aborts, traps or throws.
 *   - bf16 tensors are passed as `const void*` to 16-bit elements (upper half of an fp32).
 */
#ifndef D2MOE_H
#define D2MOE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    D2MOE_OK = 0,
    D2MOE_ERR_NULL = 1,        /* a required pointer is NULL                                  */
    D2MOE_ERR_CONFIG = 2,      /* d2moe_config is inconsistent                                */
    D2MOE_ERR_SHAPE = 3,       /* a size does not fit the configuration                       */
    D2MOE_ERR_UNSUPPORTED = 4, /* valid but not possible (e.g. D2MOE_PATH_TENSOR on an odd shape) */
    D2MOE_ERR_WORKSPACE = 5,   /* workspace or output buffer too small                        */
    D2MOE_ERR_CUDA = 6,        /* a CUDA runtime call or launch failed                        */
    D2MOE_ERR_TIMEOUT = 7,     /* device_status bit: a bounded device-side wait ran out       */
    D2MOE_ERR_NONFINITE = 8    /* device_status bit: a router logit was NaN or infinite       */
} d2moe_status;

/* bits set in *device_status */
#define D2MOE_DEV_NONFINITE 0x1  /* a router logit or an activation row held a NaN or an infinity (the
                                    outputs of such a row are zero), or an intermediate left fp16's range */
#define D2MOE_DEV_TIMEOUT   0x2
#define D2MOE_DEV_BAD_INDEX 0x4  /* a supplied routing index was out of range and was skipped */

/* kernel_path values */
#define D2MOE_PATH_AUTO      0   /* tensor-core grouped kernels where the shape allows          */
#define D2MOE_PATH_CUDA_CORE 1   /* plain fp32 CUDA-core kernels (any supported shape)          */
#define D2MOE_PATH_TENSOR    2   /* tcgen05 grouped kernels; D2MOE_ERR_UNSUPPORTED if not possible */

#define D2MOE_MAX_DIM 262144      /* largest d_model / d_ffn */
#define D2MOE_MAX_TOKENS 1048576  /* largest T of one call   */

/*
 * One MoE layer.  Candidate widths {b_k} of Section 3.3.1 are `bits[0..n_bits-1]`, ascending,
 * 1 <= bits[0], bits[n_bits-1] <= 8; every expert matrix is stored once at the top width and read
 * at any listed width (the nested store).  `group_size` is g of Eq. 2 (groups run along the input
 * dimension of each matrix) and must be a multiple of 32.  Experts are SwiGLU FFNs without bias:
 * gate and up projections [d_ffn, d_model], down projection [d_model, d_ffn].  d_model and d_ffn are
 * at most D2MOE_MAX_DIM, a call takes at most D2MOE_MAX_TOKENS tokens (D2MOE_ERR_CONFIG /
 * D2MOE_ERR_SHAPE otherwise, before anything is launched).
 */
typedef struct {
    int32_t d_model, d_ffn, n_experts, top_k, n_shared, group_size;
    int32_t n_bits, bits[8];
    int32_t renormalize;   /* 1: weights of the selected experts are divided by their sum       */
    int32_t scale_mode;    /* 0: tied residual scales s_j = s1 / 2^(j+1) (the b-bit code is then a uniform
                              b-bit grid).  1: free scales, as Eq. 4 / Eq. 5 print them: every extra bit
                              has its own fp16 scale per (row, group), s_j = mean |residual| of the group
                              (the minimiser of Eq. 5 without calibration data); the codes stay nested.
                              With free scales every batch size runs on the fp16 grouped GEMM (or the
                              CUDA-core path): the 8-bit decode kernel needs the tied form.            */
    int32_t kernel_path;   /* D2MOE_PATH_*                                                      */
    int32_t reserved[3];   /* must be 0                                                         */
} d2moe_config;

const char* d2moe_status_string(d2moe_status s);

/* Checks a configuration on the host. */
d2moe_status d2moe_check_config(const d2moe_config* cfg);

/*
 * Size in bytes of the packed form of one [rows, cols] matrix (cols % group_size == 0).
 * total = header + code bytes + metadata bytes; code_bytes and meta_bytes (either may be NULL) give
 * the split: code_bytes = rows_padded*cols*bits[n_bits-1]/8 for every width list (a width step of 3, 5,
 * 6 or 7 bits is stored as fields of 2+1, 4+1, 4+2, 4+2+1 bits), metadata = one (fp16 scale, fp16 offset)
 * pair per row and group, plus, with scale_mode 1, one fp16 scale per extra bit (bits[n_bits-1] -
 * bits[0] of them) per row and group.  The nested store costs the top width only, whatever n_bits is.
 */
d2moe_status d2moe_packed_bytes(const d2moe_config* cfg, int64_t rows, int64_t cols,
                                size_t* total_bytes, size_t* code_bytes, size_t* meta_bytes);

/*
 * MWQ quantization and packing of one matrix (Section 3.3.1: Eq. 2 base step at bits[0], then one
 * binary residual step of Eq. 4 per extra bit up to bits[n_bits-1], scales per cfg->scale_mode,
 * calibration-free).
 *   W       device, fp32 [rows, cols] row-major, finite, |W| < 65504
 *   packed  device, packed_bytes >= d2moe_packed_bytes(); 256-byte aligned; layout is private to
 *           this library (bit-plane segments tiled for the expert kernels) and versioned by a header.
 * The b-bit code of a weight is the b most significant bits of its top-width code.
 */
d2moe_status d2moe_pack_mwq(const d2moe_config* cfg, const float* W, int64_t rows, int64_t cols,
                            void* packed, size_t packed_bytes, void* stream);

/*
 * Calibration-aware MWQ (Section 3.3.1: Eq. 5 with activation statistics, Algorithm 1), scale_mode 1 only.
 *   W           device fp32 [rows, cols]; OVERWRITTEN (it is the working copy Algorithm 1 updates)
 *   hc          device fp32 [cols, cols] row-major, the upper-triangular Cholesky factor H^c of
 *               (2 X X^T + lambda I)^-1 that Algorithm 1 starts from (the caller factorises; NULL: no
 *               error compensation)
 *   col_energy  device fp32 [cols], second moment of every input column of the calibration activations
 *               (NULL: equal energies): Eq. 5 with the cross-column terms of X X^T dropped, i.e. every
 *               step's scale is the energy-weighted mean of |residual| over the group
 * Blocks are the quantization groups, left to right: a group is quantized through all its steps, its error at
 * the top width, column j divided by H^c[j, j], is taken out of all later columns (W[:, later] -= E H^c[block,
 * later]); block-level compensation only, as the paper states.  The printed loop nest of Algorithm 1 is garbled;
 * this reading is the library's.  With hc diagonal or NULL and col_energy NULL the result equals d2moe_pack_mwq.
 * Packed layout, readers and kernels are those of scale_mode 1.
 */
d2moe_status d2moe_pack_mwq_calibrated(const d2moe_config* cfg, float* W, int64_t rows, int64_t cols,
                                       const float* hc, const float* col_energy, void* packed,
                                       size_t packed_bytes, void* stream);

/*
 * Test hook: canonical codes of a packed matrix at width `bits` (bits[0] <= bits <= top width, need
 * not be a listed width): codes[r*cols + c] = top-width code >> (top - bits), one byte per weight.
 * scale / offset (either may be NULL): device fp32 [rows, cols/group_size], the stored s1 and lo.
 */
d2moe_status d2moe_unpack_codes(const d2moe_config* cfg, const void* packed, int64_t rows,
                                int64_t cols, int bits, uint8_t* codes, float* scale, float* offset,
                                void* stream);

/*
 * Test hook for scale_mode 1: the free scale of every residual step of Eq. 4, s_extra[(r * (cols /
 * group_size) + G) * n_steps + j - 1] = s_j of row r, group G, n_steps = bits[n_bits-1] - bits[0]
 * (device fp32, values are fp16-representable).  D2MOE_ERR_CONFIG when cfg->scale_mode != 1.
 */
d2moe_status d2moe_unpack_scales(const d2moe_config* cfg, const void* packed, int64_t rows, int64_t cols,
                                 float* s_extra, void* stream);

/* Workspace (device bytes) d2moe_route and d2moe_moe_forward need for up to max_tokens tokens. */
size_t d2moe_workspace_bytes(const d2moe_config* cfg, int64_t max_tokens);

/*
 * Dual routing of T tokens (Section 3.2; the models of Section 5.1) and grouping by
 * (expert, width): the histogram of the grouping is B_{j,k} of Section 3.4.3.
 * Inputs (device): x bf16 [T, d_model]; exactly one of gate_w (bf16 [E, d_model]) and logits
 * (fp32 [T, E]); exactly one of bit_w (bf16 [E, n_bits, d_model], one linear bit-width router per
 * expert) and forced_bit_idx (int8 [T, top_k], a width index per selected expert).
 * Outputs (device, all required):
 *   topk_idx  int32 [T, top_k]  selected experts, by descending logit, ties to the lower index
 *   topk_w    fp32  [T, top_k]  softmax weight of each (renormalised if cfg->renormalize)
 *   bit_idx   int8  [T, top_k]  width index: argmax of the expert's bit-width router, ties to the
 *                               lower width
 *   perm      int32 [T*top_k]   sorted position -> assignment id a = t*top_k + slot; assignments
 *                               are sorted by (expert, width index), then by a (stable)
 *   inv_perm  int32 [T*top_k]   assignment id -> sorted position
 *   group_off int32 [E*n_bits+1] exclusive prefix sum of the (expert, width) histogram
 * Logits are fp32 sums in a fixed order (32 strided partial sums of fused multiply-adds, then a
 * butterfly reduction), so the integer outputs are reproducible bit for bit.
 */
d2moe_status d2moe_route(const d2moe_config* cfg, int64_t T,
                         const void* x_bf16, const void* gate_w_bf16, const float* logits,
                         const void* bit_w_bf16, const int8_t* forced_bit_idx,
                         int32_t* topk_idx, float* topk_w, int8_t* bit_idx,
                         int32_t* perm, int32_t* inv_perm, int32_t* group_off,
                         int32_t* device_status, void* workspace, size_t workspace_bytes,
                         void* stream);

/*
 * d2moe_route without a workspace argument (the paper has no counterpart: this is an integration
 * aid).  Some callers may not allocate device memory at the point where they route a batch: a
 * serving loop whose memory pool is frozen after start-up, a plug-in that runs inside another
 * framework's step and must not touch its allocator, a component working under a fixed memory
 * budget.  For them the scratch that routing needs (sort keys and the (expert, width) histogram) is
 * a fixed array inside the library: (D2MOE_STATIC_MAX_ASSIGNMENTS + D2MOE_STATIC_MAX_KEYS) * 4
 * bytes = 72 KiB of device memory that every GPU loading the library holds until the process exits.  The call itself allocates nothing (no
 * cudaMalloc, no cudaFree, no allocating library routine).
 *   - Limits: T * top_k <= D2MOE_STATIC_MAX_ASSIGNMENTS and n_experts * n_bits <=
 *     D2MOE_STATIC_MAX_KEYS; anything larger is refused with D2MOE_ERR_WORKSPACE before any launch.
 *   - The first call on each device looks up the array's device address (with that device current)
 *     and remembers it for the life of the process; make that first call outside any stream capture.
 *     cudaDeviceReset (or any other teardown of the device's primary context) invalidates the remembered
 *     address: do not call this entry point on that device afterwards.
 *   - All calls on a device share the one array.  Calls that may overlap on the GPU (different
 *     streams, or graphs replayed concurrently) race on it and give wrong routing; serialise them.
 *     Nothing needs clearing between calls: every scratch word is written before it is read.
 * Inputs, outputs, rounding and error reporting are those of d2moe_route.
 */
#define D2MOE_STATIC_MAX_ASSIGNMENTS 16384
#define D2MOE_STATIC_MAX_KEYS 2048
d2moe_status d2moe_route_static_scratch(const d2moe_config* cfg, int64_t T,
                                        const void* x_bf16, const void* gate_w_bf16, const float* logits,
                                        const void* bit_w_bf16, const int8_t* forced_bit_idx,
                                        int32_t* topk_idx, float* topk_w, int8_t* bit_idx,
                                        int32_t* perm, int32_t* inv_perm, int32_t* group_off,
                                        int32_t* device_status, void* stream);

typedef struct {
    const void* gate_w_bf16;        /* device bf16 [E, d_model] or NULL */
    const float* logits;            /* device fp32 [T, E] or NULL       */
    const void* bit_w_bf16;         /* device bf16 [E, n_bits, d_model] or NULL */
    const int8_t* forced_bit_idx;   /* device int8 [T, top_k] or NULL   */
} d2moe_route_in;

typedef struct {                    /* outputs of an earlier d2moe_route on the same stream */
    const int32_t* topk_idx; const float* topk_w; const int8_t* bit_idx;
    const int32_t* perm; const int32_t* inv_perm; const int32_t* group_off;
} d2moe_route_out;

/*
 * The whole layer: y_t = sum over selected experts of w * Expert_{e,b}(x_t), each expert run on its
 * weights dequantized at the routed width b (Fig. 1; Section 3.3.1 reconstruction rule), plus the
 * shared experts (always on, top width, weight 1).  Expert_{e,b}(x) = Wd_b (silu(Wg_b x) * (Wu_b x)).
 *   x_bf16    device bf16 [T, d_model]
 *   expert_w  HOST array of 3*(n_experts+n_shared) device pointers to packed matrices, order
 *             [expert][gate, up, down], shared experts last; read during the call only
 *   in        routing inputs (see d2moe_route); ignored when `pre` is given
 *   pre       optional: routing already computed by d2moe_route (same T, same stream order)
 *   y_bf16    device bf16 [T, d_model], overwritten
 * Arithmetic.  Decode-sized loads (at most 40 tokens per expert on average): the packed codes are
 * multiplied as they are, as unsigned 8-bit integers, with the activations quantised per token to 15-bit
 * integers against the token's largest element (int32 accumulation; scales and offsets of Eq. 2 applied to
 * the accumulators in fp32).  That quantisation adds at most sqrt(n) / 56000 of an output's rms (n = length
 * of the dot product), whatever the spread of magnitudes inside the token.  Larger loads: weights
 * dequantized to fp16 in registers (the "dequantized to FP16" of Section 3.3.1), every token row scaled by
 * a power of two of its own so that tokens of any bf16 magnitude fit the fp16 products, h = silu(g) * u
 * stored as fp16 at the square of that scale, fp32 accumulation.  The CUDA-core path is fp32 throughout.
 * Output: bf16, round to nearest even.  A token row that holds a NaN or an infinity gives a zero output
 * row and D2MOE_DEV_NONFINITE; so does an h beyond fp16 even at its token's scale (that element is taken
 * as zero).  An index of `pre` that is out of range (expert, width index, or a position outside its
 * group) makes its assignment contribute nothing and raises D2MOE_DEV_BAD_INDEX.  T == 0 is a no-op.
 */
d2moe_status d2moe_moe_forward(const d2moe_config* cfg, int64_t T, const void* x_bf16,
                               const void* const* expert_w, const d2moe_route_in* in,
                               const d2moe_route_out* pre, void* y_bf16, int32_t* device_status,
                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * d2moe_moe_forward with timing marks for profiling: `stage_events` is a HOST array of
 * D2MOE_N_STAGES + 1 cudaEvent_t handles created by the caller with timing enabled; the call records
 * event i on `stream` before stage i and the last one after the final stage, so the caller can read
 * each stage's device time with cudaEventElapsedTime after synchronising.  Stages: 0 routing and
 * grouping (nothing when `pre` is given), 1 gate/up projection + SwiGLU, 2 down projection,
 * 3 weighted combine.  Results are identical to d2moe_moe_forward.
 */
#define D2MOE_N_STAGES 4
d2moe_status d2moe_moe_forward_events(const d2moe_config* cfg, int64_t T, const void* x_bf16,
                                      const void* const* expert_w, const d2moe_route_in* in,
                                      const d2moe_route_out* pre, void* y_bf16, int32_t* device_status,
                                      void* workspace, size_t workspace_bytes, void* stream,
                                      void* const* stage_events);

/* Number of kernel launches one d2moe_moe_forward call enqueues for T tokens (0 on a bad config), for a
 * call that passes gate weights; with more than 16 experts a call that passes logits instead makes one
 * launch fewer. */
int d2moe_forward_launch_count(const d2moe_config* cfg, int64_t T, int routing_precomputed);

/*
 * One layer of the FFN-only stack used by the multi-layer benchmark configuration (not in the
 * paper): x <- bf16( x + MoE( bf16( x / sqrt(mean(x^2) + eps) ) ) ), unit gain.  x_bf16 is updated
 * in place; xn_bf16 is a caller-provided bf16 [T, d_model] scratch that receives the normalised
 * input.  Other arguments as d2moe_moe_forward.
 */
d2moe_status d2moe_stack_layer(const d2moe_config* cfg, int64_t T, void* x_bf16, void* xn_bf16,
                               float eps, const void* const* expert_w, const d2moe_route_in* in,
                               int32_t* device_status, void* workspace, size_t workspace_bytes,
                               void* stream);

/*
 * Self-test of the bounded waits of the expert kernels.  Every wait of those kernels (on a shared-memory
 * barrier that a copy, a tensor-core operation or another warp completes) gives up after one second,
 * raises D2MOE_DEV_TIMEOUT in *device_status, and lets the kernel drain and exit, so that a lost
 * signal costs one call, not the context.  This call launches one small block that waits on a barrier
 * nothing ever completes - with the wait of the decode kernel (which = 0) or of the grouped-GEMM kernel
 * (which = 1) - and then issues a second wait, which must return at once because the block's abort flag
 * is set.  Asynchronous on the stream; takes about one second of device time; after it *device_status
 * has D2MOE_DEV_TIMEOUT set and the device is usable as before.  device_status: device int32, required.
 */
d2moe_status d2moe_selftest_wait_expiry(int which, int32_t* device_status, void* stream);

/*
 * ---- Host-side planning of the bit-width-aware I/O-compute pipeline (Section 3.4) ----
 * For deployments where the experts do not all stay in GPU memory (on one B200 they do; the layer kernels
 * above never need this).  Plain host functions: no kernel, no device memory, every array is the caller's.
 *
 * With the nested store an expert is loaded segment by segment: segment k holds what width bits[k] adds
 * to width bits[k-1]; a request at width index k reads segments 0..k.  B is the host matrix B_{j,k} of
 * Section 3.4.3, row-major [n_experts][n_bits]: requests of expert j at width index k in this layer (the
 * histogram of d2moe_route's group_off).
 */
typedef struct { int32_t expert, segment; } d2moe_plan_item;
#define D2MOE_PLAN_HEBF  0   /* Hottest-Expert-Bit-First */
#define D2MOE_PLAN_BY_ID 1   /* sequential baseline: ascending expert id, ascending width */

/*
 * Load order of the segments one layer needs (for every expert with a request: segments 0..its largest
 * requested width index).  D2MOE_PLAN_HEBF (Section 3.4.3, "Solution"): one queue per expert in ascending
 * width; the head with the highest frequency is taken next, frequency of (j, k) = requests that read
 * segment k of expert j = sum over k' >= k of B[j][k'], ties to the lower expert id.  Every expert's
 * segments appear in ascending width (constraint 6b).  queue: caller array of `capacity` items
 * (n_experts * n_bits always suffices; D2MOE_ERR_WORKSPACE if too small); *n_items receives the length.
 */
d2moe_status d2moe_plan_load_order(int32_t n_experts, int32_t n_bits, const int32_t* B, int32_t policy,
                                   d2moe_plan_item* queue, int32_t capacity, int32_t* n_items);

/*
 * The two-queue pipeline of Eq. 6 for a given load order: loads run back to back, item s taking
 * t_io[segment]; the compute of item s (its B[j][k] requests, t_comp[k] each) starts when both its load
 * (constraint 6a) and the compute of item s-1 have finished; the time the compute queue stood idle is
 * T_wait (constraint 6c).  t_io, t_comp: host double [n_bits] (the offline profile of Section 3.4.2).
 * *makespan: when both queues are done; *wait (may be NULL): summed T_wait.  An order that loads a
 * segment before the one below it is rejected (D2MOE_ERR_SHAPE).
 */
d2moe_status d2moe_plan_simulate(int32_t n_experts, int32_t n_bits, const int32_t* B,
                                 const d2moe_plan_item* queue, int32_t n_items, const double* t_io,
                                 const double* t_comp, double* makespan, double* wait);

/*
 * One layer step of the memory-budget scheduler (Algorithm 2).  `resident`: segments now in GPU memory,
 * `need`: segments the coming layer needs, `budget`: M in bytes.  Needed segments that are resident stay;
 * the others are loaded after enough other segments have been released - highest width first, then the
 * oldest layer, then the lowest expert id ("high bit-width expert weights are released ... low bit-width
 * weights are also released as needed").  Outputs (caller arrays of `capacity` entries each): the new
 * resident list, the loads and the releases.  D2MOE_ERR_WORKSPACE if the layer's own segments exceed the
 * budget or an output array is too small.
 */
typedef struct { int32_t layer, expert, segment, reserved; int64_t bytes; } d2moe_segment;
d2moe_status d2moe_plan_budget_step(const d2moe_segment* resident, int32_t n_resident,
                                    const d2moe_segment* need, int32_t n_need, int64_t budget,
                                    d2moe_segment* new_resident, int32_t* n_new,
                                    d2moe_segment* loads, int32_t* n_loads,
                                    d2moe_segment* evictions, int32_t* n_evictions, int32_t capacity);

#ifdef __cplusplus
}
#endif
#endif /* D2MOE_H */
