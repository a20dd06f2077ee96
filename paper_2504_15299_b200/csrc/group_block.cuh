// Grouping of the assignments by (expert, width) key in one launch: histogram, exclusive scan and stable scatter.
// Shared by the routing kernels and by the decode path's unit build (which runs it in front of its own work for
// decode-sized loads, so that the two need one launch instead of two).
#pragma once
#include <stdint.h>
#include <stddef.h>

// Every block stages all keys in shared memory and counts every key itself (a key per warp at a time), so no block
// waits for another; block `block` of `n_blocks` then writes the groups of the keys block, block + n_blocks, ...
// One warp per key, ballot compaction: stable.  s_grp: ((A + 31) & ~31) + n_keys + 1 ints of shared memory.  All
// threads of the block must call it; it ends with the block's last writes issued (no barrier after them).
__device__ __forceinline__ void group_block_body(int A, int n_keys, const int32_t* __restrict__ keys,
                                                 int32_t* __restrict__ group_off, int32_t* __restrict__ perm,
                                                 int32_t* __restrict__ inv_perm, int32_t* s_grp, int block, int n_blocks) {
    int32_t* s_keys = s_grp;
    int32_t* s_off = s_grp + ((A + 31) & ~31);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    for (int a = threadIdx.x; a < A; a += blockDim.x) s_keys[a] = keys[a];
    __syncthreads();
    for (int key = warp; key < n_keys; key += n_warps) {
        int cnt = 0;
        for (int base = 0; base < A; base += 32) {
            const int a = base + lane;
            cnt += __popc(__ballot_sync(0xffffffffu, a < A && s_keys[a] == key));
        }
        if (lane == 0) s_off[key] = cnt;
    }
    __syncthreads();
    if (warp == 0) {
        int carry = 0;
        for (int base = 0; base < n_keys; base += 32) {
            const int i = base + lane;
            const int v = i < n_keys ? s_off[i] : 0;
            int incl = v;
            for (int off = 1; off < 32; off <<= 1) {
                const int o = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += o;
            }
            if (i < n_keys) {
                s_off[i] = carry + incl - v;
                if (block == 0) group_off[i] = carry + incl - v;
            }
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) {
            s_off[n_keys] = carry;
            if (block == 0) group_off[n_keys] = carry;
        }
    }
    __syncthreads();
    // this block's keys, spread over its warps
    for (int key = block + warp * n_blocks; key < n_keys; key += n_warps * n_blocks) {
        int pos = s_off[key];
        if (pos == s_off[key + 1]) continue;
        for (int base = 0; base < A; base += 32) {
            const int a = base + lane;
            const bool m = a < A && s_keys[a] == key;
            const unsigned bal = __ballot_sync(0xffffffffu, m);
            if (m) {
                const int p = pos + __popc(bal & ((1u << lane) - 1u));
                perm[p] = a;
                inv_perm[a] = p;
            }
            pos += __popc(bal);
        }
    }
}

// The same grouping for one block and up to a few thousand assignments on up to 512 keys, in time proportional to
// the assignments instead of keys x assignments: a stable counting sort.  Warp w owns the contiguous chunk
// [w C, (w + 1) C) of the assignments; it walks the chunk 32 at a time, finds with one match instruction which lanes
// hold the same key and gives every assignment its rank among its warp's earlier assignments of that key
// (hist[w][key] is the running count).  A pass over (key, warp) then turns the counts into offsets: key-major, warps
// in order inside a key, so the final position = group offset + warp offset + rank is the stable one.
// s_sort: ((A + 31) & ~31) * 2 + n_warps * n_keys + n_keys + 1 ints of shared memory.  All threads of the block call
// it; blockDim.x a multiple of 32; it ends with the block's last writes issued (no barrier after them).
__host__ __device__ __forceinline__ size_t group_sort_smem_ints(int A, int n_keys, int n_warps) {
    return (size_t)((A + 31) & ~31) * 2 + (size_t)n_warps * n_keys + n_keys + 1;
}
__device__ __forceinline__ void group_sort_body(int A, int n_keys, const int32_t* __restrict__ keys,
                                                int32_t* __restrict__ group_off, int32_t* __restrict__ perm,
                                                int32_t* __restrict__ inv_perm, int32_t* s_sort) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const int A32 = (A + 31) & ~31;
    int32_t* s_keys = s_sort;                      // [A32]
    int32_t* s_rank = s_sort + A32;                // [A32] rank of an assignment among its warp's earlier ones of its key
    int32_t* hist = s_rank + A32;                  // [n_warps][n_keys]
    int32_t* s_off = hist + n_warps * n_keys;      // [n_keys + 1]
    for (int a = threadIdx.x; a < A; a += blockDim.x) s_keys[a] = keys[a];
    for (int i = threadIdx.x; i < n_warps * n_keys; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    const int C = (((A + n_warps - 1) / n_warps) + 31) & ~31;      // chunk per warp, whole 32s
    int32_t* my_hist = hist + warp * n_keys;
    for (int base = warp * C; base < min(A, (warp + 1) * C); base += 32) {
        const int a = base + lane;
        const bool live = a < A;
        const int key = live ? s_keys[a] : -1 - lane;              // dead lanes match nobody
        const unsigned same = __match_any_sync(0xffffffffu, key);
        const int rank = __popc(same & ((1u << lane) - 1u));
        int before = 0;
        if (live) before = my_hist[key];
        __syncwarp();
        if (live) {
            s_rank[a] = before + rank;
            if (rank == 0) my_hist[key] = before + __popc(same);
        }
        __syncwarp();
    }
    __syncthreads();
    // counts -> offsets of a warp's run inside its key; the key's total
    for (int key = threadIdx.x; key < n_keys; key += blockDim.x) {
        int run = 0;
        for (int w = 0; w < n_warps; ++w) {
            const int t = hist[w * n_keys + key];
            hist[w * n_keys + key] = run;
            run += t;
        }
        s_off[key] = run;
    }
    __syncthreads();
    if (warp == 0) {                               // exclusive scan of the totals
        int carry = 0;
        for (int base = 0; base < n_keys; base += 32) {
            const int i = base + lane;
            const int v = i < n_keys ? s_off[i] : 0;
            int incl = v;
            for (int off = 1; off < 32; off <<= 1) {
                const int o = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += o;
            }
            if (i < n_keys) {
                s_off[i] = carry + incl - v;
                group_off[i] = carry + incl - v;
            }
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) {
            s_off[n_keys] = carry;
            group_off[n_keys] = carry;
        }
    }
    __syncthreads();
    for (int a = threadIdx.x; a < A; a += blockDim.x) {
        const int key = s_keys[a];
        const int p = s_off[key] + hist[(a / C) * n_keys + key] + s_rank[a];
        perm[p] = a;
        inv_perm[a] = p;
    }
}
