// Block-level streaming top-k on 64-bit keys in shared memory.
//
// A key is (order-preserving score bits << 32) | payload; smaller key = better result, and all keys
// of one selection are distinct because payloads are.  Candidates that beat the current threshold
// are appended to a buffer; when the buffer could overflow, the cooperating threads sort it and
// keep the k smallest, which also tightens the threshold.  Rejecting a key only when it is larger
// than the k-th smallest key of some subset of the candidates keeps the final top-k exact.
#pragma once
#include "common.cuh"

namespace rago {

// Ascending bitonic sort of n keys (n a power of two) by `nthreads` threads; sync() is the barrier
// those threads share.  Ends with a barrier.
template <class Sync>
__device__ __forceinline__ void block_bitonic_sort(unsigned long long* keys, int n, int tid, int nthreads,
                                                   Sync sync) {
    for (int size = 2; size <= n; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int i = tid; i < (n >> 1); i += nthreads) {
                const int lo = 2 * i - (i & (stride - 1));
                const int hi = lo + stride;
                const bool up = (lo & size) == 0;
                const unsigned long long a = keys[lo], b = keys[hi];
                if ((a > b) == up) {
                    keys[lo] = b;
                    keys[hi] = a;
                }
            }
            sync();
        }
    }
}

// Sort the *cnt buffered keys ascending and cut the buffer to at most k entries.
// Must be called by all cooperating threads, after a barrier that made *cnt and the keys visible.
// Returns the new count; ends with a barrier.
template <class Sync>
__device__ __forceinline__ int block_select(unsigned long long* keys, int* cnt, int k, int tid, int nthreads,
                                            Sync sync, int cap = TOPK_CAP) {
    int n = *cnt;
    if (n > cap) n = cap;
    int n2 = 2;
    while (n2 < n) n2 <<= 1;
    for (int i = n + tid; i < n2; i += nthreads) keys[i] = KEY_MAX;
    sync();
    block_bitonic_sort(keys, n2, tid, nthreads, sync);
    const int kept = n < k ? n : k;
    if (tid == 0) *cnt = kept;
    sync();
    return kept;
}

// Ascending sort of n2 <= 64 keys (n2 a power of two) in shared memory by ONE warp, in registers: lane L holds
// elements L and L + 32 and the bitonic network's exchanges are shuffles, so no step waits on shared memory.
__device__ __forceinline__ unsigned long long shfl_xor_u64(unsigned long long v, int m) {
    const uint32_t lo = __shfl_xor_sync(0xffffffffu, (uint32_t)v, m);
    const uint32_t hi = __shfl_xor_sync(0xffffffffu, (uint32_t)(v >> 32), m);
    return ((unsigned long long)hi << 32) | lo;
}
__device__ __forceinline__ void warp_bitonic_sort(unsigned long long* keys, int n2, int lane) {
    unsigned long long k0 = lane < n2 ? keys[lane] : KEY_MAX;
    unsigned long long k1 = lane + 32 < n2 ? keys[lane + 32] : KEY_MAX;
    const int top = n2 > 32 ? 64 : 32;  // padding keys are maximal, so sorting more slots than n2 is harmless
    for (int size = 2; size <= top; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            if (stride == 32) {  // size 64: element L against element L + 32, ascending
                if (k0 > k1) { const unsigned long long t = k0; k0 = k1; k1 = t; }
            } else {
                const bool lower = (lane & stride) == 0;
                const unsigned long long o0 = shfl_xor_u64(k0, stride);
                const bool min0 = lower == ((lane & size) == 0);
                k0 = (min0 == (k0 < o0)) ? k0 : o0;
                if (top == 64) {
                    const unsigned long long o1 = shfl_xor_u64(k1, stride);
                    const bool min1 = lower == (((lane + 32) & size) == 0);
                    k1 = (min1 == (k1 < o1)) ? k1 : o1;
                }
            }
        }
    }
    if (lane < n2) keys[lane] = k0;
    if (lane + 32 < n2) keys[lane + 32] = k1;
    __syncwarp();
}
constexpr int WARP_SORT_MAX = 64;
constexpr int RANK_MAX = 256;      // block_select_short ranks up to this many keys (buffers of at least twice as many)
// Ascending sort of one 32-bit value per lane across the warp (bitonic network on shuffles); lane L returns the
// L-th smallest.
__device__ __forceinline__ uint32_t warp_sort_u32(uint32_t v, int lane) {
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const uint32_t o = __shfl_xor_sync(0xffffffffu, v, stride);
            const bool keep_min = ((lane & stride) == 0) == ((lane & size) == 0);
            v = keep_min == (v < o) ? v : o;
        }
    }
    return v;
}

// block_select for short buffers: at most WARP_SORT_MAX keys.  With at least eight warps the keys are ranked, not
// sorted: warp w counts, for each of its few keys, how many of the (distinct) keys are smaller (two votes), keeps
// key and rank in registers across one barrier and then stores the key at its rank: two barriers and a few dozen
// instructions per warp, where a bitonic network on shuffles is several hundred dependent ones in a single warp.
// Same contract as block_select.
template <class Sync>
__device__ __forceinline__ int block_select_short(unsigned long long* keys, int* cnt, int k, int tid, int nthreads,
                                                  Sync sync, int cap = TOPK_CAP) {
    int n = *cnt;
    if (n > cap) n = cap;
    const int kept = n < k ? n : k;
    if (n > WARP_SORT_MAX) {
        if (n > RANK_MAX || cap < 2 * RANK_MAX || nthreads < 256) return block_select(keys, cnt, k, tid, nthreads, sync, cap);
        // Up to RANK_MAX keys are ranked too: a lane holds every 32nd key in registers, a warp takes the keys one
        // after the other, counts the smaller ones with one compare per register and a warp-wide sum, and stores
        // the key at its rank in the free part of the buffer; three barriers where the bitonic network has dozens.
        const int warp = tid >> 5, lane = tid & 31, nwarps = nthreads >> 5;
        unsigned long long a[RANK_MAX / 32];
#pragma unroll
        for (int j = 0; j < RANK_MAX / 32; ++j) a[j] = lane + 32 * j < n ? keys[lane + 32 * j] : KEY_MAX;
        for (int i = warp; i < n; i += nwarps) {  // uniform within the warp
            const unsigned long long x = keys[i];
            uint32_t c = 0;
#pragma unroll
            for (int j = 0; j < RANK_MAX / 32; ++j) c += a[j] < x ? 1u : 0u;
            c = __reduce_add_sync(0xffffffffu, c);
            if (lane == 0 && (int)c < kept) keys[RANK_MAX + c] = x;  // keys [0, n) are only read here
        }
        sync();
        for (int i = tid; i < kept; i += nthreads) keys[i] = keys[RANK_MAX + i];
        if (tid == 0) *cnt = kept;
        sync();
        return kept;
    }
    if (nthreads >= 256) {  // uniform
        constexpr int PER_WARP = WARP_SORT_MAX / 8;
        const int warp = tid >> 5, lane = tid & 31, nwarps = nthreads >> 5;
        const unsigned long long a = lane < n ? keys[lane] : KEY_MAX;
        const unsigned long long b = lane + 32 < n ? keys[lane + 32] : KEY_MAX;
        unsigned long long mine[PER_WARP];
        int rank[PER_WARP];
#pragma unroll
        for (int t = 0; t < PER_WARP; ++t) {
            const int i = warp + t * nwarps;
            rank[t] = -1;
            mine[t] = 0ull;
            if (i < n) {  // uniform within the warp
                const unsigned long long x = keys[i];
                rank[t] = __popc(__ballot_sync(0xffffffffu, a < x)) + __popc(__ballot_sync(0xffffffffu, b < x));
                mine[t] = x;
            }
        }
        sync();  // every key has been read
        if (lane == 0) {
#pragma unroll
            for (int t = 0; t < PER_WARP; ++t)
                if (rank[t] >= 0 && rank[t] < kept) keys[rank[t]] = mine[t];
        }
        if (tid == 0) *cnt = kept;
        sync();
        return kept;
    }
    if (tid < 32) {
        int n2 = 2;
        while (n2 < n) n2 <<= 1;
        for (int i = n + tid; i < n2; i += 32) keys[i] = KEY_MAX;
        __syncwarp();
        warp_bitonic_sort(keys, n2, tid);
        if (tid == 0) *cnt = kept;
    }
    sync();
    return kept;
}

// Append `key` for the lanes with pred set; one shared atomic per warp.  Whole warp must call.
__device__ __forceinline__ void warp_push(unsigned long long* keys, int* cnt, bool pred, unsigned long long key,
                                          int cap = TOPK_CAP) {
    const unsigned mask = __ballot_sync(0xffffffffu, pred);
    if (mask == 0) return;
    const int lane = threadIdx.x & 31;
    const int leader = __ffs(mask) - 1;
    int base = 0;
    if (lane == leader) base = atomicAdd(cnt, __popc(mask));
    base = __shfl_sync(0xffffffffu, base, leader);
    if (pred) {
        const int idx = base + __popc(mask & ((1u << lane) - 1u));
        if (idx < cap) keys[idx] = key;
    }
}

}  // namespace rago
