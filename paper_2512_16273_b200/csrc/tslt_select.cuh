// Bitonic sort of 64-bit keys in shared memory by the 256 threads of a CTA.
#pragma once

#include "tslt_common.cuh"

namespace tslt {

// Sorts a[0..P) (P a power of two), descending if kDescending.  All 256 threads call it.
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

}  // namespace tslt
