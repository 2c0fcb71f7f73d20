// Exact selection primitives for the 256 consumer threads of a CTA, all on shared memory:
// radix select of the r-th largest / smallest 32-bit value of a filtered array, trimming a
// candidate buffer to its exact top-k under the order (key descending, index ascending),
// and a bitonic sort of 64-bit keys.
#pragma once

#include "tslt_common.cuh"

namespace tslt {

struct SelectScratch {
    uint32_t hist[256];
    int bin;
    int above;
    int counter;
    int pad;
};

// r-th (1-based) largest (kLargest) or smallest value among { get(i) : 0 <= i < n, pred(i) },
// examined over the bytes [lo_byte, hi_byte] of the value (other bytes are known to agree for
// all members, their common bits passed in `fixed`).  Returns the value; *n_before gets the
// number of members strictly before it in the chosen direction.  Requires 1 <= r <= #members.
template <bool kLargest, typename Get, typename Pred>
__device__ __forceinline__ uint32_t radix_select(int n, int r, int hi_byte, int lo_byte, uint32_t fixed,
                                                 Get get, Pred pred, SelectScratch* sc, int tid,
                                                 int* n_before) {
    uint32_t prefix = fixed, mask = 0;
    int remaining = r, before = 0;
    for (int byte = hi_byte; byte >= lo_byte; --byte) {
        const int shift = byte * 8;
        sc->hist[tid] = 0;
        consumer_sync();
        for (int i = tid; i < n; i += kConsumerThreads) {
            if (pred(i)) {
                uint32_t v = get(i);
                if ((v & mask) == (prefix & mask)) atomicAdd(&sc->hist[(v >> shift) & 255u], 1u);
            }
        }
        consumer_sync();
        if (tid < 32) {
            // lane l owns 8 consecutive bins in walking order (descending bins for kLargest)
            uint32_t c[8];
            uint32_t tot = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                int w = tid * 8 + j;  // walking position 0..255
                int b = kLargest ? 255 - w : w;
                c[j] = sc->hist[b];
                tot += c[j];
            }
            uint32_t incl = tot;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
                if (tid >= o) incl += t;
            }
            uint32_t excl = incl - tot;
            if (excl < (uint32_t)remaining && (uint32_t)remaining <= incl) {
                uint32_t run = excl;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (run < (uint32_t)remaining && (uint32_t)remaining <= run + c[j]) {
                        int w = tid * 8 + j;
                        sc->bin = kLargest ? 255 - w : w;
                        sc->above = (int)run;
                    }
                    run += c[j];
                }
            }
        }
        consumer_sync();
        const int bin = sc->bin, above = sc->above;
        before += above;
        remaining -= above;
        prefix = (prefix & ~(255u << shift)) | ((uint32_t)bin << shift);
        mask |= 255u << shift;
    }
    consumer_sync();
    *n_before = before;
    return prefix;
}

// Candidate buffer: (key, idx) pairs, unordered.
struct Candidates {
    uint32_t* key;
    int* idx;
    uint32_t* tmp_key;  // k entries
    int* tmp_idx;       // k entries
    int* count;         // shared counter
};

// Exact top-k, under the order (key descending, idx ascending), of a virtual sequence of n
// items; item i is a member iff src.valid(i) and has src.key(i), src.idx(i) (indices are
// distinct).  The winners replace the contents of the candidate buffer (the source may read the
// buffer: winners are staged in tmp first).  All 256 consumer threads call it with the same
// arguments after a barrier.  Returns true iff at least k members exist, in which case
// *kth_key is the k-th key; *cb.count is set to min(k, members).
// kKeyHiOnly: keys come from bf16 values, so only the two high bytes vary (the low 16 bits
// follow from the sign).  idx_hi_byte: highest byte of an index that can be non-zero.
template <bool kKeyHiOnly, typename Src>
__device__ __forceinline__ bool select_topk(const Src& src, int n, int k, int idx_hi_byte, Candidates cb,
                                            SelectScratch* sc, int tid, uint32_t* kth_key) {
    int* iscr = reinterpret_cast<int*>(sc->hist);
    int my = 0;
    for (int i = tid; i < n; i += kConsumerThreads) my += src.valid(i) ? 1 : 0;
    const int members = block_sum_int(my, tid, iscr);
    uint32_t kth = 0, idx_cut = 0xffffffffu;
    const bool full = members >= k;
    if (members > k) {
        int n_gt;
        auto valid = [&](int i) { return src.valid(i); };
        auto getk = [&](int i) { return src.key(i); };
        if (kKeyHiOnly) {
            kth = radix_select<true>(n, k, 3, 2, 0u, getk, valid, sc, tid, &n_gt);
            // low half of a key made from a bf16 value: 0x0000 for non-negative, 0xffff for negative
            kth = (kth & 0xffff0000u) | ((kth & 0x80000000u) ? 0u : 0xffffu);
        } else {
            kth = radix_select<true>(n, k, 3, 0, 0u, getk, valid, sc, tid, &n_gt);
        }
        const int need = k - n_gt;  // ties to keep, >= 1
        int eq = 0;
        for (int i = tid; i < n; i += kConsumerThreads) eq += (src.valid(i) && src.key(i) == kth) ? 1 : 0;
        const int n_eq = block_sum_int(eq, tid, iscr);
        if (n_eq > need) {
            int dummy;
            auto tie = [&](int i) { return src.valid(i) && src.key(i) == kth; };
            auto geti = [&](int i) { return (uint32_t)src.idx(i); };
            idx_cut = radix_select<false>(n, need, idx_hi_byte, 0, 0u, geti, tie, sc, tid, &dummy);
        }
    } else if (members == k) {
        // the k-th key is the smallest member
        uint32_t mn = 0xffffffffu;
        for (int i = tid; i < n; i += kConsumerThreads)
            if (src.valid(i)) mn = min(mn, src.key(i));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mn = min(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        if ((tid & 31) == 0) sc->hist[tid >> 5] = mn;
        consumer_sync();
        mn = sc->hist[0];
#pragma unroll
        for (int w = 1; w < kConsumerWarps; ++w) mn = min(mn, sc->hist[w]);
        consumer_sync();
        kth = mn;
    }
    *kth_key = kth;
    if (tid == 0) sc->counter = 0;
    consumer_sync();
    for (int i = tid; i < n; i += kConsumerThreads) {
        if (!src.valid(i)) continue;
        const uint32_t key = src.key(i);
        const int id = src.idx(i);
        if (key > kth || (key == kth && (uint32_t)id <= idx_cut)) {
            const int pos = atomicAdd(&sc->counter, 1);
            if (pos < k) {
                cb.tmp_key[pos] = key;
                cb.tmp_idx[pos] = id;
            }
        }
    }
    consumer_sync();
    const int kept = min(sc->counter, k);
    for (int i = tid; i < kept; i += kConsumerThreads) {
        cb.key[i] = cb.tmp_key[i];
        cb.idx[i] = cb.tmp_idx[i];
    }
    consumer_sync();
    if (tid == 0) *cb.count = kept;
    consumer_sync();
    return full;
}

// Bitonic sort of a[0..P) (P a power of two, shared memory), descending if kDescending.
template <bool kDescending>
__device__ __forceinline__ void bitonic_sort(unsigned long long* a, int P, int tid) {
    for (int size = 2; size <= P; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int i = tid; i < (P >> 1); i += kConsumerThreads) {
                int lo = 2 * i - (i & (stride - 1));
                int hi = lo + stride;
                bool up = ((lo & size) == 0);  // first half of each bitonic block
                unsigned long long x = a[lo], y = a[hi];
                bool swap = kDescending ? (up ? x < y : x > y) : (up ? x > y : x < y);
                if (swap) {
                    a[lo] = y;
                    a[hi] = x;
                }
            }
            consumer_sync();
        }
    }
}

__device__ __forceinline__ int next_pow2(int n) {
    int p = 1;
    while (p < n) p <<= 1;
    return p;
}

}  // namespace tslt
