// Block-wide exact top-k selection (multi-class radix select) and ordered stream
// compaction.  Used by the per-event key-token top-k, the event-weighted top-k of
// the prefill pruning step and the KV TOPK policy.
//
// Ordering: item i outranks item j when its score is larger, or equal with i < j.
// Both are folded into one 64-bit key, key64 = float_key(score) << 32 | ~i, so
// "the n best of class g" is exactly { i : key64(i) >= thr[g] } for one threshold.
#pragma once

#include "common.cuh"

namespace metok {

struct SelectSmem {
    unsigned long long prefix[METOK_MAX_GROUPS];  // bits of the threshold fixed so far
    int need[METOK_MAX_GROUPS];                   // items still to take among the undecided ones
    int pop[METOK_MAX_GROUPS];                    // class population
    int eq[METOK_MAX_GROUPS];                     // items in the threshold's bin of the last pass
    int live[METOK_MAX_GROUPS];                   // class still needs a threshold search
    int warp_tot[32];
    int carry;
};

__device__ __forceinline__ unsigned long long key64_of(float score, int i) {
    return ((unsigned long long)float_key(score) << 32) | (unsigned long long)(~(uint32_t)i);
}

// Adds 1 to bins[slot] for every active lane, one atomic per distinct slot in the warp.
__device__ __forceinline__ void warp_aggregated_inc(uint32_t* bins, int slot, bool active) {
    const unsigned mask = __ballot_sync(0xFFFFFFFFu, active);
    if (active) {
        const unsigned peers = __match_any_sync(mask, slot);
        if ((int)(threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&bins[slot], __popc(peers));
    }
}

// Finds thr[g] for every class.  `hist` is G*256 uint32 of shared memory.
// cls(i) -> class in [0,G) or -1 (item takes no part); val(i) -> score.
// budget[g] >= 0 is clamped to the class population.
// After the call: selected(i) <=> sm.need[g] > 0 && key64(i) >= sm.prefix[g]   (need restored to the clamped budget)
template <typename ClsF, typename ValF>
__device__ void block_select_thresholds(int n, int G, ClsF cls, ValF val, const int* budget,
                                        uint32_t* hist, SelectSmem& sm, int* clamped_budget /*smem [G]*/) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int n_round = (n + 31) & ~31;   // whole warps enter the aggregated atomics together
    for (int g = tid; g < G; g += nthr) { sm.pop[g] = 0; }
    __syncthreads();
    if (G == 1) {
        // population of a single class: count the participating items
        int c = 0;
        for (int i = tid; i < n; i += nthr) c += (cls(i) == 0);
        c = warp_sum_int(c);
        if ((tid & 31) == 0 && c) atomicAdd(&sm.pop[0], c);
    } else {
        for (int i = tid; i < n_round; i += nthr) {
            const int g = (i < n) ? cls(i) : -1;
            warp_aggregated_inc(reinterpret_cast<uint32_t*>(sm.pop), g < 0 ? 0 : g, g >= 0);
        }
    }
    __syncthreads();
    for (int g = tid; g < G; g += nthr) {
        int b = budget[g];
        b = b < sm.pop[g] ? b : sm.pop[g];
        clamped_budget[g] = b;
        sm.need[g] = b;
        sm.prefix[g] = 0ull;
        sm.eq[g] = 0;
        // nothing to search when the class keeps none or all of its items
        sm.live[g] = (b > 0 && b < sm.pop[g]) ? 1 : 0;
    }
    __syncthreads();

    for (int pass = 0; pass < 8; ++pass) {
        const int shift = 56 - 8 * pass;
        int any_live = 0;
        for (int g = 0; g < G; ++g) any_live |= sm.live[g];
        if (!any_live) break;
        for (int b = tid; b < G * 256; b += nthr) hist[b] = 0u;
        __syncthreads();
        for (int i = tid; i < n_round; i += nthr) {
            bool act = false;
            int slot = 0;
            if (i < n) {
                const int g = cls(i);
                if (g >= 0 && sm.live[g]) {
                    const unsigned long long k = key64_of(val(i), i);
                    const unsigned long long pf = sm.prefix[g];
                    const bool match = (pass == 0) || ((k >> (shift + 8)) == (pf >> (shift + 8)));
                    if (match) { act = true; slot = g * 256 + (int)((k >> shift) & 255ull); }
                }
            }
            warp_aggregated_inc(hist, slot, act);
        }
        __syncthreads();
        for (int g = tid; g < G; g += nthr) {
            if (!sm.live[g]) continue;
            int cum = 0;
            const int want = sm.need[g];
            for (int b = 255; b >= 0; --b) {
                const int c = (int)hist[g * 256 + b];
                if (cum + c >= want) {
                    sm.need[g] = want - cum;
                    sm.prefix[g] |= ((unsigned long long)b) << shift;
                    sm.eq[g] = c;
                    break;
                }
                cum += c;
            }
            // every undecided item in the bin is taken: the remaining bits can stay 0
            if (sm.eq[g] == sm.need[g]) sm.live[g] = 0;
        }
        __syncthreads();
    }
    for (int g = tid; g < G; g += nthr) {
        sm.need[g] = clamped_budget[g];
        if (clamped_budget[g] >= sm.pop[g]) sm.prefix[g] = 0ull;   // keep all
    }
    __syncthreads();
}

// Ordered compaction: for i in [0,n) in ascending order, emit(i, rank) for every
// flagged i, rank counting flagged items before it.  Returns the total (valid in
// every thread).
template <typename FlagF, typename EmitF>
__device__ int block_compact(int n, FlagF flag, EmitF emit, SelectSmem& sm) {
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5;
    const int nwarps = nthr >> 5;
    if (tid == 0) sm.carry = 0;
    __syncthreads();
    for (int base = 0; base < n; base += nthr) {
        const int i = base + tid;
        const bool f = (i < n) && flag(i);
        const unsigned bal = __ballot_sync(0xFFFFFFFFu, f);
        const int in_warp = __popc(bal & ((1u << lane) - 1u));
        if (lane == 0) sm.warp_tot[warp] = __popc(bal);
        __syncthreads();
        int before = 0, total = 0;
        for (int w = 0; w < nwarps; ++w) {
            const int c = sm.warp_tot[w];
            if (w < warp) before += c;
            total += c;
        }
        const int carry = sm.carry;
        if (f) emit(i, carry + before + in_warp);
        __syncthreads();
        if (tid == 0) sm.carry = carry + total;
        __syncthreads();
    }
    return sm.carry;
}

}  // namespace metok
