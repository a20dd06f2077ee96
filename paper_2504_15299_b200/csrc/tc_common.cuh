// Device-side building blocks shared by the tensor-core expert kernels: mbarrier, bulk-copy / TMA,
// tcgen05 (MMA, TMEM load/store, commit, fences), operand descriptors; host-side tensor maps.
#pragma once
#include "d2moe_common.cuh"

#include <cuda.h>

struct TmaMaps { CUtensorMap m[5]; };  // box heights 16, 32, 64, 128, 256 rows x 64 fp16 columns

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// try_wait with a suspend-time hint: the warp sleeps in hardware (issuing nothing) until the phase
// completes or about `ns` nanoseconds pass, instead of spinning through the issue slots and the
// integer pipe that the working warps need.
__device__ __forceinline__ bool mbar_try_sleep(uint32_t bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(ns) : "memory");
    return ok != 0;
}
// true in exactly one lane of a converged warp
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  `abort_flag` (shared) is set by the first wait that runs out (about one second);
// once it is set no wait blocks any more, so the CTA drains and exits instead of hanging.  The loop
// lives in a function of its own: the waits are inlined dozens of times and the hot loops of the
// expert kernels are bound by instruction fetch, so only the first try is inline.
static __device__ __noinline__ void mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status, bool drain) {
    unsigned long long t0 = 0;
    for (unsigned spin = 0;; ++spin) {
        if (mbar_try_sleep(bar, parity, 4000u)) return;
        if ((spin & 15u) == 15u) {
            if (*abort_flag && !drain) return;      // a drain wait keeps its own one-second limit
            const unsigned long long now = globaltimer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > 1000000000ull) {
                *abort_flag = 1;
                if (status) atomicOr(status, D2MOE_DEV_TIMEOUT);
                return;
            }
        }
    }
}
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                          bool drain = false) {
    if (mbar_try(bar, parity)) return;
    mbar_wait_slow(bar, parity, abort_flag, status, drain);
}

// The same bounded wait written entirely in PTX: the common case (phase already complete) costs the
// try_wait and one predicated branch, with no integer instructions to turn the predicate into a
// value and back.  abort_addr: shared-memory address of the CTA's abort flag; status must not be null.
__device__ __forceinline__ void mbar_wait_ptx(uint32_t bar, uint32_t parity, uint32_t abort_addr, int32_t* status) {
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        ".reg .u32 ab;\n\t"
        ".reg .u64 t0, t1;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%0], %1;\n\t"
        "@p bra WAIT_DONE;\n\t"
        "mov.u64 t0, %%globaltimer;\n"
        "WAIT_RETRY:\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%0], %1, 4000;\n\t"
        "@p bra WAIT_DONE;\n\t"
        "ld.volatile.shared.u32 ab, [%2];\n\t"
        "setp.ne.u32 q, ab, 0;\n\t"
        "@q bra WAIT_DONE;\n\t"
        "mov.u64 t1, %%globaltimer;\n\t"
        "sub.u64 t1, t1, t0;\n\t"
        "setp.lt.u64 q, t1, 1000000000;\n\t"
        "@q bra WAIT_RETRY;\n\t"
        "st.volatile.shared.u32 [%2], 1;\n\t"
        "red.global.or.b32 [%3], 2;\n"    // D2MOE_DEV_TIMEOUT
        "WAIT_DONE:\n\t"
        "}"
        ::"r"(bar), "r"(parity), "r"(abort_addr), "l"(status) : "memory");
}

// The same for kernels whose barrier block is 512-byte aligned and keeps the abort flag at byte 504 and
// the device-status pointer at byte 496 of that block: the slow path finds both from the barrier's own
// address, so a wait keeps no register alive besides the barrier address and the parity.
__device__ __forceinline__ void mbar_wait_blk(uint32_t bar, uint32_t parity) {
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        ".reg .u32 ab, blk;\n\t"
        ".reg .u64 t0, t1, st;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%0], %1;\n\t"
        "@p bra WAITB_DONE;\n\t"
        "and.b32 blk, %0, 0xFFFFFE00;\n\t"
        "mov.u64 t0, %%globaltimer;\n"
        "WAITB_RETRY:\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%0], %1, 4000;\n\t"
        "@p bra WAITB_DONE;\n\t"
        "ld.volatile.shared.u32 ab, [blk+504];\n\t"
        "setp.ne.u32 q, ab, 0;\n\t"
        "@q bra WAITB_DONE;\n\t"
        "mov.u64 t1, %%globaltimer;\n\t"
        "sub.u64 t1, t1, t0;\n\t"
        "setp.lt.u64 q, t1, 1000000000;\n\t"
        "@q bra WAITB_RETRY;\n\t"
        "st.volatile.shared.u32 [blk+504], 1;\n\t"
        "ld.shared.u64 st, [blk+496];\n\t"
        "red.global.or.b32 [st], 2;\n"    // D2MOE_DEV_TIMEOUT
        "WAITB_DONE:\n\t"
        "}"
        ::"r"(bar), "r"(parity) : "memory");
}

__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem descriptor]; fp16 inputs, fp32 accumulation
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// the same with the shared-memory descriptor given as two 32-bit halves (its high word is a constant)
__device__ __forceinline__ void tc_mma_ts_lohi(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 bd;\n\tsetp.ne.b32 p, %5, 0;\n\tmov.b64 bd, {%2, %3};\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], bd, %4, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                 ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
                   "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]) : "memory");
}
__device__ __forceinline__ void tc_st8(uint32_t taddr, const uint32_t (&v)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]) : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// K-major, 128-byte-swizzled shared-memory operand: 8-row atoms of 1024 bytes.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);         // start address
    d |= (uint64_t)1 << 16;                           // leading byte offset (unused with swizzle)
    d |= (uint64_t)(1024 >> 4) << 32;                 // stride byte offset: next 8-row atom
    d |= (uint64_t)1 << 46;                           // descriptor version
    d |= (uint64_t)2 << 61;                           // 128B swizzle
    return d;
}
// fp16 x fp16 -> fp32, A and B K-major, M = 128
__device__ __forceinline__ uint32_t instr_desc_f16(int n) {
    return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

__device__ __forceinline__ __half2 h2dup(float v) { return __float2half2_rn(v); }
__device__ __forceinline__ __half2 as_h2(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }
__device__ __forceinline__ uint32_t as_u32(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }

// Compile-time description of a width list of at most four widths: nibble j of WPACK is the width of step j
// (bits[j] - bits[j-1]; sw: the width of the field it is stored in when that is a single field).  WPACK == 0
// selects the run-time path.
template <int WPACK>
struct WidthList {
    __host__ __device__ static constexpr int w(int j) { return (WPACK >> (4 * j)) & 15; }
    __host__ __device__ static constexpr int sw(int j) { return w(j) <= 1 ? 1 : (w(j) <= 2 ? 2 : (w(j) <= 4 ? 4 : 8)); }
    __host__ __device__ static constexpr int count() { int k = 0; while (k < 8 && w(k) != 0) ++k; return k; }
    __host__ __device__ static constexpr int top() { int b = 0; for (int i = 0; i < count(); ++i) b += w(i); return b; }
    __host__ __device__ static constexpr int pos(int j) { int b = 0; for (int i = 0; i <= j; ++i) b += w(i); return top() - b; }
    // a step of w bits is stored as power-of-two fields that add up to exactly w bits per code
    __host__ __device__ static constexpr int seg_off(int gs, int j) { int o = D2MOE_TILE_ROWS * 4; for (int i = 0; i < j; ++i) o += D2MOE_TILE_ROWS * gs * w(i) / 8; return o; }
};

// exponent S of the common factor 2^-S from the header of a packed matrix
__device__ __forceinline__ int matrix_exponent(const uint8_t* packed) {
    const PackHeader* h = reinterpret_cast<const PackHeader*>(packed);
    const float s1max = __uint_as_float(h->s1_max_bits);
    const float wabs = __uint_as_float(h->wabs_max_bits) + 4.0f * s1max;
    int e1, e2;
    frexpf(s1max, &e1);            // s1max = m * 2^e1, 0.5 <= m < 1  =>  s1max <= 2^e1
    frexpf(wabs, &e2);
    int S = e1 + 9;                // s1max * 2^(24 - S) <= 2^15
    if (e2 - 15 > S) S = e2 - 15;  // |tile| <= 2^15
    return S;
}


// ------------------------------------------------------------------------------------------------
// Host: tensor maps over a row-major fp16 [rows, cols] buffer, 128-byte swizzle, boxes of 64 columns
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static inline EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn) return fn;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
        return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
    return fn;
}

// ------------------------------------------------------------------------------------------------
// Host: per-process caches, so that a layer call does not repeat driver queries whose answer cannot change
// ------------------------------------------------------------------------------------------------
// number of SMs of the current device
static inline int device_sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int sms = 148;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cached[dev] = sms;
    }
    return cached[dev];
}

// raises the dynamic shared-memory limit of kernel Kern on the current device when a launch needs more than
// any earlier one did (the attribute is per device and sticks)
template <auto Kern>
static inline cudaError_t ensure_dynamic_smem(int bytes) {
    static int set[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
    if (set[dev] >= bytes) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(Kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) set[dev] = bytes;
    return e;
}

// the tensor maps of the last few (buffer, shape) pairs this thread built: a serving loop calls with the same
// workspace every step, so its maps are encoded once
struct TmaMapCacheEntry { const void* base; long long rows, cols; int kind, dev; TmaMaps maps; };
template <typename Build>
static inline bool cached_maps(TmaMaps* out, int kind, void* base, long long rows, long long cols, Build build) {
    static thread_local TmaMapCacheEntry cache[8];
    static thread_local int next = 0, used = 0;
    int dev = 0;
    cudaGetDevice(&dev);
    for (int i = 0; i < used; ++i) {
        const TmaMapCacheEntry& c = cache[i];
        if (c.base == base && c.rows == rows && c.cols == cols && c.kind == kind && c.dev == dev) { *out = c.maps; return true; }
    }
    if (!build(out)) return false;
    TmaMapCacheEntry& c = cache[next];
    c.base = base; c.rows = rows; c.cols = cols; c.kind = kind; c.dev = dev; c.maps = *out;
    next = (next + 1) & 7;
    if (used < 8) ++used;
    return true;
}

static inline bool make_maps_uncached(TmaMaps* maps, void* base, long long rows, long long cols) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return false;
    for (int i = 0; i < 5; ++i) {
        cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
        cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
        cuuint32_t box[2] = {64, (cuuint32_t)(16 << i)};
        cuuint32_t estr[2] = {1, 1};
        if (enc(&maps->m[i], CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, base, dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return false;
    }
    return true;
}

static inline bool make_maps(TmaMaps* maps, void* base, long long rows, long long cols) {
    return cached_maps(maps, 0, base, rows, cols, [&](TmaMaps* m) { return make_maps_uncached(m, base, rows, cols); });
}
