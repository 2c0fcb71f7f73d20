// The bulk-copy ring that streams one row segment from HBM through shared memory:
// a producer warp issues one untiled TMA copy per tile and signals a "full" mbarrier;
// eight consumer warps each own a 2 KB chunk of every tile and release the slot through an
// "empty" mbarrier.  Every wait is bounded; a wait that runs out raises an abort flag that
// all roles poll, and sets the status word of the workspace.
#pragma once

#include "tslt_common.cuh"

namespace tslt {

struct RingBars {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    int abort;
    int pad;
};

__device__ __forceinline__ void ring_init(RingBars* bars, int tid) {
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], kConsumerWarps);
        }
        bars->abort = 0;
        mbar_fence_init();
    }
}

__device__ __forceinline__ void raise_abort(RingBars* bars, int* ws_status) {
    bars->abort = 1;
    atomicOr(ws_status, kStatusWaitTimeout);
}

// Producer warp: tiles [tile_begin, tile_end) of a row of row_bytes bytes starting at `row`.
// The last tile of the row may be ragged: its 16-byte-aligned part is bulk-copied, the
// remaining < 16 bytes are copied with plain loads and the vector is padded with -inf.
template <typename T>
__device__ __forceinline__ void producer_loop(const unsigned char* row, long long row_bytes, int tile_begin,
                                              int tile_end, unsigned char* ring, RingBars* bars,
                                              int* ws_status) {
    const int lane = threadIdx.x & 31;
    const uint64_t policy = l2_evict_first_policy();
    int issued = 0;
    for (int t = tile_begin; t < tile_end; ++t, ++issued) {
        const int s = issued % kStages, use = issued / kStages;
        if (*(volatile int*)&bars->abort) break;
        if (use > 0) {
            int ok = 1;
            if (lane == 0) ok = mbar_wait(&bars->empty[s], (uint32_t)((use - 1) & 1), &bars->abort) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) {
                if (lane == 0) raise_abort(bars, ws_status);
                break;
            }
        }
        const long long off = (long long)t * kTileBytes;
        const long long left = row_bytes - off;
        const uint32_t bytes = (uint32_t)(left < (long long)kTileBytes ? left : (long long)kTileBytes);
        const uint32_t bulk = bytes & ~15u, rem = bytes - bulk;
        unsigned char* dst = ring + s * kTileBytes;
        if (rem) {
            constexpr int per = 16 / Elt<T>::kBytes;
            if (lane < per) {
                const int valid = (int)rem / Elt<T>::kBytes;
                if (Elt<T>::kBytes == 4) {
                    uint32_t v = 0xff800000u;  // -inf
                    if (lane < valid) v = __ldg(reinterpret_cast<const uint32_t*>(row + off + bulk) + lane);
                    reinterpret_cast<uint32_t*>(dst + bulk)[lane] = v;
                } else {
                    unsigned short v = 0xff80u;  // bf16 -inf
                    if (lane < valid) v = __ldg(reinterpret_cast<const unsigned short*>(row + off + bulk) + lane);
                    reinterpret_cast<unsigned short*>(dst + bulk)[lane] = v;
                }
            }
            __syncwarp();
        }
        if (lane == 0) {
            if (bulk) {
                mbar_arrive_expect_tx(&bars->full[s], bulk);
                bulk_copy_g2s(dst, row + off, bulk, &bars->full[s], policy);
            } else {
                mbar_arrive(&bars->full[s]);
            }
        }
    }
    // The producer does not leave while one of its copies may still be in flight: it waits
    // (bounded) for the completion of the last tiles it issued, one per ring slot.
    if (lane == 0) {
        const int first = issued > kStages ? issued - kStages : 0;
        for (int i = first; i < issued; ++i) {
            bool done = false;
            for (uint32_t probe = 0; probe < kSpinLimit && !done; ++probe) {
                done = mbar_try_wait(&bars->full[i % kStages], (uint32_t)((i / kStages) & 1));
                if (!done && (probe & 63u) == 63u) __nanosleep(64);
            }
            if (!done) atomicOr(ws_status, kStatusWaitTimeout);
        }
    }
}

// Bytes of tile t that hold data after padding the ragged tail to a full 16-byte vector.
__device__ __forceinline__ uint32_t tile_padded_bytes(long long row_bytes, int t) {
    const long long left = row_bytes - (long long)t * kTileBytes;
    const uint32_t bytes = (uint32_t)(left < (long long)kTileBytes ? left : (long long)kTileBytes);
    return (bytes + 15u) & ~15u;
}

}  // namespace tslt
