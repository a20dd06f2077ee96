// Grouping of the assignments by (expert, width) key in one launch: histogram, exclusive scan and stable scatter.
// Shared by the routing kernels and by the decode path's unit build (which runs it in front of its own work for
// decode-sized loads, so that the two need one launch instead of two).
#pragma once
#include <stdint.h>

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
