// tslt_sparsify: draft-side sparsify-then-sample (Section 3, Solution 1; the sampling steps
// of Algorithms 2 and 4) as two kernels on the caller's stream.
//
// Streaming kernel.  One CTA reads one segment of one logits row from HBM exactly once, with
// 16-byte loads that go straight to registers (each warp instruction covers 512 contiguous
// bytes).  It keeps two things: each lane's online (max, sum) for the softmax normaliser, and,
// for every 64-byte tile of the row (32 bf16 or 16 fp32 logits), the top 16 bits of the tile's
// largest logit, written to the workspace (2 bytes per 64 read).  Nothing in it depends on k or
// top_p: there is no threshold, no histogram, no shared memory and no barrier in the loop, so it
// runs at the occupancy and speed of a plain streaming reduction.
//
// Finish kernel (launched with programmatic stream serialization; a CTA starts on its row as soon
// as the row's segments have been handed over).  One CTA per row:
//   1. a lower bound on the k-th largest TILE maximum: tiles are taken in groups so that there are
//      a few times k groups, and the k-th largest group maximum is found by bisection on its 16
//      bits (each of the k groups at or above it holds a tile, and so a logit, at or above it);
//   2. the tiles at or above that bound are listed in address order ("survivors": a little more
//      than k of them) and read back from global memory: 64 bytes each, k * 64 bytes of the row's
//      V * e;
//   3. the exact k-th largest logit among them by a histogram over the 16-bit keys between the
//      bound and the row maximum (fp32 rows: a second histogram over the low 16 bits inside the
//      boundary value), ties at the boundary going to the lower index;
//   4. the winners are collected by prefix sums over the survivors in address order, so they come
//      out in ascending token index without any sort;
//   5. the top-rho cut (a sort of the at most k winners by logit, an fp64 cumulative), the
//      renormalised distribution and its CDF in fp64, the samples by inverse CDF, the outputs.
// A row whose survivors do not fit the list (thousands of tied tile maxima: constant rows, rows
// sorted by value) runs steps 3 and 4 over all of its vectors instead: slower, same code.
#include <math.h>

#include "tslt_common.cuh"
#include "tslt_rowmath.cuh"
#include "tslt_select.cuh"

namespace tslt {

constexpr int kTilesPerChunk = 32;        // 64-byte tiles in a 2 KB chunk
constexpr int kVecsPerTile = 4;           // 16-byte vectors in a tile
constexpr int kSparsifyStreamCtasPerSm = 6;
constexpr int kFinishThreads = kBlockThreads;
constexpr int kMaxGroups = 4096;          // group maxima the finish kernel bisects over
constexpr int kMaxTileList = 4096;        // survivor tiles it can list
constexpr int kSelBins = 1024;            // bins of the selection histogram
constexpr uint32_t kLowestFinite16 = 0x0080u;   // key of -FLT_MAX >> 16
constexpr uint32_t kHighestFinite16 = 0xff7fu;  // key of +FLT_MAX >> 16

// What a segment hands over besides its tile maxima: one (max, sum) pair per warp.
struct SegStat {
    double S[kWarps];  // sum of 2^(y - M) over the warp's chunks of the segment
    float M[kWarps];   // the warp's reference exponent (base 2)
};

struct SparsifyParams {
    const unsigned char* logits;
    long long row_stride_bytes;
    int V, rows, k;
    float top_p;
    ScaleC c;
    int num_samples;
    const float* uniforms;
    int* idx;
    float* logit;
    int* count;
    int* token;
    float* lse;
    float* mass;
    int nchunks;
    RowSplit split;
    int group_log2;   // tiles per group = 1 << group_log2
    int ngroups;      // <= kMaxGroups
    int tile_cap;     // survivor list capacity (<= kMaxTileList)
    int poll_limit;   // polls of a segment's ready flag before falling back to the end of the streaming kernel
    int* status;
    int* seg_ready;           // [rows * nseg]
    SegStat* seg_stats;       // [rows * nseg]
    unsigned short* tile_max; // [rows, nchunks * 32]: top 16 bits of each tile's largest logit, slot order (see tile_slot)
};

// Tile a of a row is its bytes [64 a, 64 a + 64).  In the streaming kernel vector j * 32 + l of a
// chunk belongs to lane l, so the tile made of vectors j * 32 + 4 q .. + 3 belongs to the lane
// quad q, whose leader stores the maxima of its four tiles (j = 0..3) side by side: slot
// ch * 32 + q * 4 + j holds tile ch * 32 + j * 8 + q.
__host__ __device__ inline int tile_slot(int a) { return (a & ~31) | ((a & 7) << 2) | ((a >> 3) & 3); }

// Order-preserving 16-bit key of the top half of an fp32 / a bf16 pattern, -0 folded onto +0
// (equal to float_to_key(value) >> 16 for the value the pattern truncates).
__device__ __forceinline__ uint32_t raw16_to_key16(uint32_t r) {
    r = (r == 0x8000u) ? 0u : r;
    return (r & 0x8000u) ? (~r & 0xffffu) : (r | 0x8000u);
}

// ---- streaming kernel ------------------------------------------------------------------------------
template <typename T> struct QuadMax;
template <> struct QuadMax<bf16_t> {
    // top 16 bits of the largest logit of each of the quad's four tiles, packed (j = 0, 1 | 2, 3)
    static __device__ __forceinline__ uint2 keys(const LaneTile<bf16_t>& lt) {
        uint32_t r[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t v = lt.vm[j];
            v = bf16x2_max(v, __shfl_xor_sync(0xffffffffu, v, 1));
            v = bf16x2_max(v, __shfl_xor_sync(0xffffffffu, v, 2));
            r[j] = bf16x2_max(v, v >> 16) & 0xffffu;
        }
        return make_uint2(r[0] | (r[1] << 16), r[2] | (r[3] << 16));
    }
};
template <> struct QuadMax<float> {
    static __device__ __forceinline__ uint2 keys(const LaneTile<float>& lt) {
        uint32_t r[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float v = lt.vm[j];
            v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
            v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
            r[j] = __float_as_uint(v) >> 16;
        }
        return make_uint2(r[0] | (r[1] << 16), r[2] | (r[3] << 16));
    }
};

template <typename T>
__global__ void __launch_bounds__(kBlockThreads, kSparsifyStreamCtasPerSm) sparsify_stream_kernel(const SparsifyParams p) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const RowWork wk = locate_work(p.split, blockIdx.x, p.nchunks);
    const unsigned char* rowp = p.logits + (long long)wk.row * p.row_stride_bytes;
    const RowExtent ext = row_extent<T>(p.V);
    const float c = p.c.f;
    const unsigned char* lane_rowp = rowp + lane * kVecBytes;
    int ch = wk.chunk_begin + warp;
    LaneTile<T> lt;
    if (ch < wk.chunk_end) lt.load_lane(lane_rowp, ch * kVecsPerChunk, ext);  // in flight during the set-up below
    // The segment's ready flag is cleared here, by the CTA that will set it, and the store is fenced
    // before the barrier after which this CTA lets the finish kernel be scheduled.  A finish CTA
    // runs only after every streaming CTA has passed that point, so it never sees a flag (or a
    // status word) left by an earlier call, and the workspace needs no clearing between calls.
    if (tid == 0) {
        *(volatile int*)&p.seg_ready[blockIdx.x] = 0;
        if (blockIdx.x == 0) *(volatile int*)p.status = 0;
        __threadfence();
    }
    __syncthreads();
    allow_dependent_launch();

    LaneSum ls;
    ls.reset();
    unsigned short* tmax = p.tile_max + (size_t)wk.row * p.nchunks * kTilesPerChunk;
    while (ch < wk.chunk_end) {
        const float lm = lt.reduce_max();
        const uint2 q = QuadMax<T>::keys(lt);
        if ((lane & 3) == 0) *reinterpret_cast<uint2*>(tmax + ch * kTilesPerChunk + lane) = q;  // slots (lane >> 2) * 4 ..+3
        ls.raise_to(lm, c);
        lt.accumulate(ls, c);
        ch += kWarps;
        if (ch < wk.chunk_end) lt.load_lane(lane_rowp, ch * kVecsPerChunk, ext);
    }
    // hand-over: one (M, S) pair per warp
    const float Mw = warp_max(ls.M);
    const double Sw = warp_sum(ls.total_f64() * exp2((double)ls.M - (double)Mw));
    if (lane == 0) {
        SegStat* st = &p.seg_stats[blockIdx.x];
        st->S[warp] = Sw;
        st->M[warp] = Mw;
    }
    __syncthreads();  // every warp's part of the hand-over is written
    if (tid == 0) publish_row_ready(&p.seg_ready[blockIdx.x]);
}

// ---- finish kernel ---------------------------------------------------------------------------------
__host__ __device__ inline size_t align16(size_t x) { return (x + 15) / 16 * 16; }
__host__ __device__ inline int pow2_at_least(int n) {
    int p = 1;
    while (p < n) p <<= 1;
    return p;
}
constexpr int kFinishHeaderBytes = 512;
// dynamic shared memory of the finish kernel: header | histogram | region A | region B | winners
__host__ __device__ inline size_t finish_region_a(int ngroups, int k) {
    const size_t g = (size_t)ngroups * 4, c = (size_t)pow2_at_least(k) * 8;
    return align16(g > c ? g : c);
}
__host__ __device__ inline size_t finish_region_b(int tile_cap, int k) {
    const size_t t = (size_t)tile_cap * 4, w = (size_t)k * 16;
    return align16(t > w ? t : w);
}
__host__ __device__ inline size_t sparsify_finish_smem(int ngroups, int tile_cap, int k) {
    return kFinishHeaderBytes + (size_t)kSelBins * 4 + finish_region_a(ngroups, k) + finish_region_b(tile_cap, k) + (size_t)k * 8;
}

struct FinishShared {
    double scratch[16];
    double lrow;            // base-2 log of the row's softmax normaliser
    int round_count[32];    // one counter per bisection round
    int iscr[16];
    int sel_bin, sel_above, sel_eq, sel_total;
    int ready, n_surv, max16;
};

// One 16-byte vector of a row as kPer logits; the row's ragged last vector element by element,
// -inf beyond the row.
template <typename T>
__device__ __forceinline__ void load_row_vector(const unsigned char* rowp, int vi, const RowExtent& ext, int V,
                                                float (&z)[Elt<T>::kPerVec]) {
    constexpr int kPer = Elt<T>::kPerVec;
    if (vi < ext.nvec_full) {
        unpack_vec<T>(__ldcg(reinterpret_cast<const uint4*>(rowp) + vi), z);
    } else {
#pragma unroll
        for (int e = 0; e < kPer; ++e) z[e] = vi * kPer + e < V ? Elt<T>::load(rowp, vi * kPer + e) : -INFINITY;
    }
}

// Exclusive prefix sum of one int per thread over the block; *total gets the sum.
__device__ __forceinline__ int block_exscan(int v, int tid, int* scr /* >= 8 */, int* total) {
    const int lane = tid & 31, warp = tid >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) scr[warp] = incl;
    consumer_sync();
    int base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        const int t = scr[w];
        if (w < warp) base += t;
        tot += t;
    }
    consumer_sync();
    *total = tot;
    return base + incl - v;
}

// Which of a chunk's 32 tiles have a key >= bound: bit a of the result is tile a of the chunk in
// ADDRESS order (tile j * 8 + q sits in slot q * 4 + j of the chunk's 64-byte line of maxima).
__device__ __forceinline__ uint32_t chunk_survivors(const unsigned short* line, uint32_t bound) {
    uint32_t w[16];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint4 v = __ldcg(reinterpret_cast<const uint4*>(line) + i);
        w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
    }
    uint32_t m = 0;
#pragma unroll
    for (int a = 0; a < kTilesPerChunk; ++a) {
        const int slot = ((a & 7) << 2) | (a >> 3);
        const uint32_t raw = (slot & 1) ? (w[slot >> 1] >> 16) : (w[slot >> 1] & 0xffffu);
        m |= (raw16_to_key16(raw) >= bound ? 1u : 0u) << a;
    }
    return m;
}

// The vectors a thread works on: units [u0, u1) of the row's survivor tiles (tl: their tile numbers in
// address order, four vectors each), or of the whole row (tl == nullptr: unit = vector).  f(z, vi)
// is called for each of them in ascending order with the vector's logits (-inf beyond the row).
template <typename T, typename F>
__device__ __forceinline__ void for_my_vectors(const unsigned char* rowp, const RowExtent& ext, int V, const uint32_t* tl,
                                               int u0, int u1, F f) {
    constexpr int kPer = Elt<T>::kPerVec;
    constexpr int kInFlight = 4;
    for (int u = u0; u < u1; u += kInFlight) {
        uint4 d[kInFlight];
        int vi[kInFlight];
#pragma unroll
        for (int i = 0; i < kInFlight; ++i) {
            const int uu = u + i;
            vi[i] = -1;
            if (uu < u1) vi[i] = tl ? (int)(tl[uu >> 2] * (uint32_t)kVecsPerTile) + (uu & 3) : uu;
            if (vi[i] >= 0 && vi[i] < ext.nvec_full) d[i] = __ldcg(reinterpret_cast<const uint4*>(rowp) + vi[i]);
        }
#pragma unroll
        for (int i = 0; i < kInFlight; ++i) {
            if (vi[i] < 0) continue;
            float z[kPer];
            if (vi[i] < ext.nvec_full) unpack_vec<T>(d[i], z);
            else load_row_vector<T>(rowp, vi[i], ext, V, z);
            f(z, vi[i]);
        }
    }
}

// The kk-th largest of the values value_of(z) in [lo, hi] over the thread block's vectors (values
// outside the range, or negative, do not take part), by a histogram of kSelBins bins over the
// range, narrowed once more if the range is wider than the histogram.  Results in sh: sel_bin = the
// value, sel_above = how many are larger (inside [lo, hi]), sel_eq = how many equal it,
// sel_total = how many lie in [lo, hi].  If fewer than kk lie in the range, sel_bin = -1 and only
// sel_total is meaningful.  All threads call it; hist is kSelBins words of shared memory.
template <typename T, typename VF>
__device__ __forceinline__ void hist_select(const unsigned char* rowp, const RowExtent& ext, int V, const uint32_t* tl, int u0,
                                            int u1, VF value_of, int lo, int hi, int kk, FinishShared* sh, uint32_t* hist,
                                            int tid) {
    constexpr int kPer = Elt<T>::kPerVec;
    int above_acc = 0, total_first = -1;
    for (;;) {
        int s = 0;
        while (((hi - lo) >> s) >= kSelBins) ++s;
        for (int i = tid; i < kSelBins; i += kFinishThreads) hist[i] = 0u;
        consumer_sync();
        for_my_vectors<T>(rowp, ext, V, tl, u0, u1, [&](const float(&z)[kPer], int) {
            int cur = -1;
            uint32_t run = 0;
#pragma unroll
            for (int e = 0; e < kPer; ++e) {
                const int v = value_of(z[e]);
                if (v >= lo && v <= hi) {
                    const int b = (v - lo) >> s;
                    if (b != cur) {  // equal neighbours (ties) cost one atomic, not one each
                        if (run) atomicAdd(&hist[cur], run);
                        cur = b;
                        run = 0;
                    }
                    ++run;
                }
            }
            if (run) atomicAdd(&hist[cur], run);
        });
        consumer_sync();
        if (tid < 32) {
            // rows of 32 bins from the top; lane l takes bin top - l of the row
            uint32_t carried = 0;
            int found_bin = -1;
            uint32_t found_above = 0, found_eq = 0;
            const int nb = ((hi - lo) >> s) + 1;
            for (int top = nb - 1; top >= 0; top -= 32) {
                const int b = top - tid;
                const uint32_t cnt = b >= 0 ? hist[b] : 0u;
                uint32_t incl = cnt;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
                    if (tid >= o) incl += t;
                }
                const unsigned hit = __ballot_sync(0xffffffffu, carried + incl >= (uint32_t)kk);
                if (hit && found_bin < 0) {
                    const int l = __ffs(hit) - 1;
                    found_bin = top - l;
                    found_above = carried + __shfl_sync(0xffffffffu, incl - cnt, l);
                    found_eq = __shfl_sync(0xffffffffu, cnt, l);
                }
                carried += __shfl_sync(0xffffffffu, incl, 31);
            }
            if (tid == 0) {
                sh->sel_bin = found_bin;
                sh->sel_above = (int)found_above;
                sh->sel_eq = (int)found_eq;
                sh->sel_total = (int)carried;
            }
        }
        consumer_sync();
        const int bin = sh->sel_bin, above = sh->sel_above, eq = sh->sel_eq, total = sh->sel_total;
        consumer_sync();
        if (total_first < 0) total_first = total;
        if (bin < 0 || s == 0) {
            if (tid == 0) {
                sh->sel_bin = bin < 0 ? -1 : lo + bin;
                sh->sel_above = above_acc + above;
                sh->sel_eq = eq;
                sh->sel_total = total_first;
            }
            consumer_sync();
            return;
        }
        above_acc += above;
        kk -= above;
        lo = lo + (bin << s);
        hi = min(hi, lo + (1 << s) - 1);
    }
}

template <typename T>
__global__ void __launch_bounds__(kFinishThreads, 4) sparsify_finish_kernel(const SparsifyParams p) {
    constexpr int kPer = Elt<T>::kPerVec;
    constexpr bool kBf16 = (Elt<T>::kBytes == 2);
    extern __shared__ __align__(128) unsigned char smem_raw[];
    // carve-up (sizes in sparsify_finish_smem): header | hist | region A | region B | win_raw | win_idx
    //   region A: group maxima, later the sort keys of the top-rho cut
    //   region B: survivor tile list, later the fp64 work arrays
    FinishShared* sh = reinterpret_cast<FinishShared*>(smem_raw);
    static_assert(sizeof(FinishShared) <= kFinishHeaderBytes, "header");
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem_raw + kFinishHeaderBytes);
    const int k = p.k;
    const size_t a_bytes = finish_region_a(p.ngroups, k), b_bytes = finish_region_b(p.tile_cap, k);
    uint32_t* gm = reinterpret_cast<uint32_t*>(smem_raw + kFinishHeaderBytes + kSelBins * 4);
    unsigned long long* comp = reinterpret_cast<unsigned long long*>(gm);
    uint32_t* tl = reinterpret_cast<uint32_t*>(smem_raw + kFinishHeaderBytes + kSelBins * 4 + a_bytes);
    double* cum = reinterpret_cast<double*>(tl);
    double* wv = cum + k;
    uint32_t* win_raw = reinterpret_cast<uint32_t*>(smem_raw + kFinishHeaderBytes + kSelBins * 4 + a_bytes + b_bytes);
    int* win_idx = reinterpret_cast<int*>(win_raw + k);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, row = blockIdx.x;
    const int nseg = p.split.nseg;
    const unsigned char* rowp = p.logits + (long long)row * p.row_stride_bytes;
    const RowExtent ext = row_extent<T>(p.V);
    if (tid == 0 && p.num_samples > 0)  // the uniforms are needed last: ask for their cache line now
        asm volatile("prefetch.global.L2 [%0];" ::"l"(p.uniforms + (size_t)row * p.num_samples));
    if (tid < 32) sh->round_count[tid] = 0;
    // ---- wait for the row's segments --------------------------------------------------------------
    // Nothing the streaming kernel wrote is read before this point.  The row's own segments being
    // handed over is enough to go on; a flag that does not come within the poll limit is recorded in
    // the status word and the CTA waits for the end of the streaming kernel instead.
    if (tid < 32) {
        bool ok = true;
        for (int s = lane; s < nseg; s += 32) ok = poll_row_ready(&p.seg_ready[(size_t)row * nseg + s], p.poll_limit) && ok;
        ok = __all_sync(0xffffffffu, ok);
        if (lane == 0) sh->ready = ok ? 1 : 0;
    }
    __syncthreads();
    if (!sh->ready) {
        if (tid == 0) atomicOr(p.status, TSLT_STATUS_WAIT_FELL_BACK);
        wait_for_primary_kernel();
    }
    __syncthreads();
    // ---- the row's log-normaliser, by one warp (fp64 is scarce) -------------------------------------
    if (warp == 1) {
        const SegStat* st = p.seg_stats + (size_t)row * nseg;
        double Mall = -INFINITY;
        for (int i = lane; i < nseg * kWarps; i += 32)
            if (__ldcg(&st[i / kWarps].S[i % kWarps]) > 0.0) Mall = fmax(Mall, (double)__ldcg(&st[i / kWarps].M[i % kWarps]));
        Mall = warp_max(Mall);
        double Sall = 0.0;
        for (int i = lane; i < nseg * kWarps; i += 32) {
            const double Sw = __ldcg(&st[i / kWarps].S[i % kWarps]);
            if (Sw > 0.0) Sall += Sw * exp2((double)__ldcg(&st[i / kWarps].M[i % kWarps]) - Mall);
        }
        Sall = warp_sum(Sall);
        if (lane == 0) sh->lrow = Sall > 0.0 ? Mall + log2(Sall) : -INFINITY;
    }
    // ---- 1. group maxima of the tile keys ---------------------------------------------------------------
    const int ntiles = p.nchunks * kTilesPerChunk;
    const unsigned short* tmax = p.tile_max + (size_t)row * ntiles;
    const int glog = p.group_log2, ngroups = p.ngroups;
    if (glog > 3)
        for (int i = tid; i < ngroups; i += kFinishThreads) gm[i] = 0u;
    if (tid == 0) sh->max16 = 0;
    __syncthreads();
    {
        uint32_t my_max = 0;
        const int nv8 = ntiles / 8;
        for (int v = tid; v < nv8; v += kFinishThreads) {
            const uint4 w = __ldcg(reinterpret_cast<const uint4*>(tmax) + v);
            uint32_t kk[8];
            kk[0] = raw16_to_key16(w.x & 0xffffu); kk[1] = raw16_to_key16(w.x >> 16);
            kk[2] = raw16_to_key16(w.y & 0xffffu); kk[3] = raw16_to_key16(w.y >> 16);
            kk[4] = raw16_to_key16(w.z & 0xffffu); kk[5] = raw16_to_key16(w.z >> 16);
            kk[6] = raw16_to_key16(w.w & 0xffffu); kk[7] = raw16_to_key16(w.w >> 16);
            // groups are runs of consecutive SLOTS (any fixed partition of the tiles will do)
            if (glog == 0) {
#pragma unroll
                for (int i = 0; i < 8; ++i) gm[v * 8 + i] = kk[i];
            } else if (glog == 1) {
#pragma unroll
                for (int i = 0; i < 4; ++i) gm[v * 4 + i] = max(kk[2 * i], kk[2 * i + 1]);
            } else if (glog == 2) {
#pragma unroll
                for (int i = 0; i < 2; ++i) gm[v * 2 + i] = max(max(kk[4 * i], kk[4 * i + 1]), max(kk[4 * i + 2], kk[4 * i + 3]));
            }
            const uint32_t m8 = max(max(max(kk[0], kk[1]), max(kk[2], kk[3])), max(max(kk[4], kk[5]), max(kk[6], kk[7])));
            if (glog == 3) gm[v] = m8;
            else if (glog > 3) atomicMax(&gm[v >> (glog - 3)], m8);
            my_max = max(my_max, m8);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) my_max = max(my_max, __shfl_xor_sync(0xffffffffu, my_max, o));
        if (lane == 0) atomicMax(&sh->max16, (int)my_max);
    }
    __syncthreads();
    const int max16 = min(sh->max16, (int)kHighestFinite16);
    const double L2 = sh->lrow;
    // ---- 2. the k-th largest group maximum, by bisection on its 16 bits -----------------------------------
    uint32_t bound = 0;
    if (ngroups >= k) {
        for (int bit = 15; bit >= 0; --bit) {
            const uint32_t cand = bound | (1u << bit);
            int cnt = 0;
            for (int i = tid; i < ngroups; i += kFinishThreads) cnt += gm[i] >= cand ? 1 : 0;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
            if (lane == 0 && cnt) atomicAdd(&sh->round_count[bit], cnt);
            __syncthreads();
            if (sh->round_count[bit] >= k) bound = cand;
        }
    }
    int lo16 = max((int)bound, (int)kLowestFinite16);
    // ---- 3. survivor tiles (key >= bound), listed in address order -----------------------------------------
    // Thread t takes a run of consecutive chunks; a chunk's 32 tile keys are one 64-byte line.
    const int cpt = (p.nchunks + kFinishThreads - 1) / kFinishThreads;
    const int ch0 = min(p.nchunks, tid * cpt), ch1 = min(p.nchunks, ch0 + cpt);
    int my_surv = 0;
    for (int ch = ch0; ch < ch1; ++ch) my_surv += __popc(chunk_survivors(tmax + ch * kTilesPerChunk, (uint32_t)lo16));
    int n_surv;
    int pos = block_exscan(my_surv, tid, sh->iscr, &n_surv);
    const bool listed = n_surv <= p.tile_cap;
    if (listed) {
        for (int ch = ch0; ch < ch1; ++ch) {
            uint32_t m = chunk_survivors(tmax + ch * kTilesPerChunk, (uint32_t)lo16);  // bit a: tile a of the chunk
            while (m) {
                const int a = __ffs(m) - 1;
                m &= m - 1;
                tl[pos++] = (uint32_t)(ch * kTilesPerChunk + a);
            }
        }
    }
    __syncthreads();
    // the vectors this thread works on from here: a contiguous run of the survivors' vectors, or of the row's
    const uint32_t* units = listed ? tl : nullptr;
    const int n_units = listed ? n_surv * kVecsPerTile : (p.V + kPer - 1) / kPer;
    const int upt = (n_units + kFinishThreads - 1) / kFinishThreads;
    const int u0 = min(n_units, tid * upt), u1 = min(n_units, u0 + upt);
    if (!listed) lo16 = (int)kLowestFinite16;

    // ---- 4. the exact k-th largest logit --------------------------------------------------------------------
    // level 1: its 16-bit key among the finite logits of the survivors
    auto key16_of = [](float z) -> int {
        const uint32_t k16 = float_to_key(z) >> 16;
        return (k16 >= kLowestFinite16 && k16 <= kHighestFinite16) ? (int)k16 : -1;
    };
    int n0 = 0;                 // winners: min(k, finite logits)
    uint32_t e32 = 0;           // key of the k-th largest logit
    int need_ties = 0;          // how many logits equal to it are winners (the lowest indices)
    if (max16 >= lo16) {
        hist_select<T>(rowp, ext, p.V, units, u0, u1, key16_of, lo16, max16, k, sh, hist, tid);
        const int e16 = sh->sel_bin, above = sh->sel_above, eq = sh->sel_eq, total = sh->sel_total;
        consumer_sync();
        if (e16 < 0) {  // fewer than k finite logits in the row: all of them win
            n0 = total;
            e32 = 0u;
            need_ties = 0;
            // every finite logit is "above" the key 0; nothing ties
        } else if (kBf16) {
            n0 = k;
            e32 = ((uint32_t)e16 << 16) | ((e16 & 0x8000) ? 0u : 0xffffu);  // keys of bf16 values: low half follows the sign
            need_ties = k - above;
        } else {
            // level 2 (fp32 rows): the low 16 bits among the logits whose high bits equal e16
            const uint32_t hi_bits = (uint32_t)e16;
            auto low16_of = [hi_bits](float z) -> int {
                const uint32_t kz = float_to_key(z);
                return (kz >> 16) == hi_bits ? (int)(kz & 0xffffu) : -1;
            };
            hist_select<T>(rowp, ext, p.V, units, u0, u1, low16_of, 0, 0xffff, k - above, sh, hist, tid);
            const int low = sh->sel_bin, above2 = sh->sel_above;
            consumer_sync();
            n0 = k;
            e32 = (hi_bits << 16) | (uint32_t)low;
            need_ties = k - above - above2;
            (void)eq;
        }
    }
    // ---- 5. the winners, in ascending index ---------------------------------------------------------------
    int n = 0;
    if (n0 > 0) {
        int c_gt = 0, c_eq = 0;
        const uint32_t e32c = e32;
        for_my_vectors<T>(rowp, ext, p.V, units, u0, u1, [&](const float(&z)[kPer], int) {
#pragma unroll
            for (int e = 0; e < kPer; ++e) {
                if (key16_of(z[e]) < lo16) continue;
                const uint32_t kz = float_to_key(z[e]);
                c_gt += kz > e32c ? 1 : 0;
                c_eq += kz == e32c ? 1 : 0;
            }
        });
        int tot_eq, tot_w;
        const int eq_before = block_exscan(c_eq, tid, sh->iscr, &tot_eq);
        const int my_ties = max(0, min(c_eq, need_ties - eq_before));
        int wpos = block_exscan(c_gt + my_ties, tid, sh->iscr, &tot_w);
        int ties_left = my_ties;
        for_my_vectors<T>(rowp, ext, p.V, units, u0, u1, [&](const float(&z)[kPer], int vi) {
#pragma unroll
            for (int e = 0; e < kPer; ++e) {
                if (key16_of(z[e]) < lo16) continue;
                const uint32_t kz = float_to_key(z[e]);
                bool win = kz > e32c;
                if (kz == e32c && ties_left > 0) {
                    win = true;
                    --ties_left;
                }
                if (win && wpos < k) {
                    win_raw[wpos] = __float_as_uint(z[e]);
                    win_idx[wpos] = vi * kPer + e;
                    ++wpos;
                }
            }
        });
        n = min(tot_w, k);
        __syncthreads();
    }
    n0 = n;
    const double cf = (double)p.c.f;  // the scale the streaming sum used: keeps q consistent with the normaliser
    const double cd = p.c.d;
    double mass = 0.0;
    // ---- 6. top-rho cut ---------------------------------------------------------------------------------------
    if (n0 > 0 && p.top_p < 1.0f) {
        const int P = pow2_at_least(n0);
        for (int i = tid; i < P; i += kFinishThreads)
            comp[i] = i < n0 ? (((unsigned long long)float_to_key(__uint_as_float(win_raw[i])) << 32) |
                                (unsigned long long)(0xffffffffu - (uint32_t)win_idx[i])) : 0ull;
        consumer_sync();
        bitonic_sort<true>(comp, P, tid);
        for (int i = tid; i < n0; i += kFinishThreads)
            cum[i] = exp2((double)key_to_float((uint32_t)(comp[i] >> 32)) * cf - L2);
        consumer_sync();
        block_inclusive_scan(cum, n0, tid, sh->scratch);
        const double tp = (double)p.top_p;
        int lo = 0, hi = n0;
        while (lo < hi) {  // first n with c_n >= top_p
            const int mid = (lo + hi) >> 1;
            if (cum[mid] >= tp) hi = mid; else lo = mid + 1;
        }
        n = lo < n0 ? lo + 1 : n0;
        mass = cum[n - 1];
        consumer_sync();
        if (n < n0) {
            // keep what precedes the cut in (logit descending, index ascending): a larger key, or the
            // cut's key and an index up to the cut's
            const unsigned long long cutc = comp[n - 1];
            const uint32_t ckey = (uint32_t)(cutc >> 32);
            const int cidx = (int)(0xffffffffu - (uint32_t)cutc);
            const int ipt = (n0 + kFinishThreads - 1) / kFinishThreads;
            const int i0 = min(n0, tid * ipt), i1 = min(n0, i0 + ipt);
            uint32_t keep_raw[4];
            int keep_idx[4];
            int kept = 0;
            for (int i = i0; i < i1; ++i) {  // ipt <= 4 (k <= 1024)
                const uint32_t kz = float_to_key(__uint_as_float(win_raw[i]));
                if (kz > ckey || (kz == ckey && win_idx[i] <= cidx)) {
                    keep_raw[kept] = win_raw[i];
                    keep_idx[kept] = win_idx[i];
                    ++kept;
                }
            }
            int tot;
            int kp = block_exscan(kept, tid, sh->iscr, &tot);  // (its barriers order the reads above before the writes below)
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (i < kept) {
                    win_raw[kp + i] = keep_raw[i];
                    win_idx[kp + i] = keep_idx[i];
                }
            consumer_sync();
        }
    }
    // ---- 7. renormalised truncated distribution in fp64, CDF, samples, outputs ----------------------------
    double my_max = -INFINITY;
    for (int i = tid; i < n; i += kFinishThreads) {
        const double y = (double)__uint_as_float(win_raw[i]) * cd;
        wv[i] = y;
        my_max = fmax(my_max, y);
    }
    const double mS = block_max(my_max, tid, sh->scratch);
    double my_mass = 0.0;
    for (int i = tid; i < n; i += kFinishThreads) {
        if (!(p.top_p < 1.0f)) my_mass += exp2((double)__uint_as_float(win_raw[i]) * cf - L2);
        const double w = exp2(wv[i] - mS);
        wv[i] = w;
        cum[i] = w;
    }
    if (!(p.top_p < 1.0f)) mass = block_sum(my_mass, tid, sh->scratch);
    else consumer_sync();
    block_inclusive_scan(cum, n, tid, sh->scratch);

    int* o_idx = p.idx + (size_t)row * k;
    float* o_logit = p.logit + (size_t)row * k;
    for (int i = tid; i < k; i += kFinishThreads) {
        o_idx[i] = i < n ? win_idx[i] : -1;
        o_logit[i] = i < n ? __uint_as_float(win_raw[i]) : -INFINITY;
    }
    if (tid == 0) {
        p.count[row] = n;
        if (p.lse) p.lse[row] = n0 > 0 ? (float)(L2 * 0.6931471805599453) : -INFINITY;
        if (p.mass) p.mass[row] = n0 > 0 ? (float)mass : 0.f;
    }
    const double W = n > 0 ? cum[n - 1] : 0.0;
    for (int sidx = tid; sidx < p.num_samples; sidx += kFinishThreads) {
        int tok = -1;
        if (n > 0) {
            const float u = clamp_uniform(p.uniforms[(size_t)row * p.num_samples + sidx]);
            int pos2 = first_greater(cum, n, (double)u * W);
            if (pos2 >= n) {
                pos2 = n - 1;
                while (pos2 > 0 && !(wv[pos2] > 0.0)) --pos2;
            }
            tok = win_idx[pos2];
        }
        p.token[(size_t)row * p.num_samples + sidx] = tok;
    }
    // this kernel's completion must imply the streaming kernel's (what follows on the stream relies
    // on it): one CTA sees to that; the others leave and make room
    if (row == 0) wait_for_primary_kernel();
}

}  // namespace tslt

// ---- host side -------------------------------------------------------------------------------
namespace tslt {

struct SparsifyPlan {
    int nchunks, group_log2, ngroups, tile_cap;
    RowSplit split;
    size_t fin_smem;
    size_t ws_ready_off, ws_stats_off, ws_tiles_off, ws_bytes;
};

static int sm_count_cached() {
    static int sms = 0;
    if (sms == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 148;
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
        sms = v;
    }
    return sms;
}

static SparsifyPlan make_sparsify_plan(int rows, int V, int k, int elt_bytes) {
    SparsifyPlan pl;
    const long long row_bytes = (long long)V * elt_bytes;
    pl.nchunks = (int)((row_bytes + kChunkBytes - 1) / kChunkBytes);
    const long long ntiles = (long long)pl.nchunks * kTilesPerChunk;
    // tiles per group: the largest power of two that still leaves 2 k groups (the k-th largest group
    // maximum is then a selective bound), and no more groups than the finish kernel holds
    int glog = 0;
    while ((ntiles >> (glog + 1)) >= 2LL * k) ++glog;
    while (((ntiles + (1LL << glog) - 1) >> glog) > kMaxGroups) ++glog;
    pl.group_log2 = glog;
    pl.ngroups = (int)((ntiles + (1LL << glog) - 1) >> glog);
    pl.tile_cap = 8 * k < 512 ? 512 : (8 * k > kMaxTileList ? kMaxTileList : 8 * k);
    pl.fin_smem = sparsify_finish_smem(pl.ngroups, pl.tile_cap, k);
    // One CTA per row when the rows fill the machine; fewer rows are cut into segments (at least one
    // chunk per warp each) so that every CTA slot has work.  A segment costs nothing but its own
    // hand-over (8 (max, sum) pairs and a flag).
    const int slots = kSparsifyStreamCtasPerSm * sm_count_cached();
    int nseg = 1;
    if (rows > 0 && rows < slots) {
        nseg = (slots + rows - 1) / rows;
        const int by_len = pl.nchunks / kWarps;
        if (nseg > by_len) nseg = by_len;
        if (nseg > 64) nseg = 64;
        if (nseg < 1) nseg = 1;
    }
    int cps = (pl.nchunks + nseg - 1) / nseg;
    if (cps < 1) cps = 1;
    pl.split.rows = rows;
    pl.split.cps = cps;
    pl.split.nseg = (pl.nchunks + cps - 1) / cps;
    pl.split.grid = rows * pl.split.nseg;
    size_t off = kWsHeaderBytes;
    pl.ws_ready_off = off;
    off = align_up256(off + (size_t)rows * pl.split.nseg * sizeof(int));
    pl.ws_stats_off = off;
    off = align_up256(off + (size_t)rows * pl.split.nseg * sizeof(SegStat));
    pl.ws_tiles_off = off;
    off = align_up256(off + (size_t)rows * (size_t)ntiles * sizeof(unsigned short));
    pl.ws_bytes = off;
    return pl;
}

ScaleC make_scale(float temperature) {
    const double c = 1.4426950408889634 / (double)temperature;
    ScaleC s;
    s.f = (float)c;
    s.d = c;
    return s;
}

// Polls of a ready flag before a finish CTA gives up on it (about a second at 200 ns per poll).
static int g_sparsify_poll_limit = kReadyPollLimit;

}  // namespace tslt

using namespace tslt;

extern "C" int tslt_sparsify_workspace_bytes(int rows, int V, int k, int num_samples, size_t* bytes) {
    if (!bytes || rows < 0 || V <= 0 || k <= 0 || k > V || k > TSLT_MAX_K || num_samples < 0)
        return TSLT_ERR_INVALID_ARG;
    SparsifyPlan a = make_sparsify_plan(rows, V, k, 2), b = make_sparsify_plan(rows, V, k, 4);
    *bytes = a.ws_bytes > b.ws_bytes ? a.ws_bytes : b.ws_bytes;
    return TSLT_OK;
}

extern "C" int tslt_set_ready_poll_limit(int polls) {
    if (polls < 0) return TSLT_ERR_INVALID_ARG;
    g_sparsify_poll_limit = polls;
    return TSLT_OK;
}

extern "C" int tslt_sparsify(const void* logits, int dtype, int B, int gamma, int V,
                             long long row_stride_elems, int k, float top_p, float temperature,
                             int num_samples, const float* uniforms, int* idx, float* logit, int* count,
                             int* token, float* lse, float* mass, void* workspace, size_t workspace_bytes,
                             void* stream) {
    if (dtype != TSLT_F32 && dtype != TSLT_BF16) return TSLT_ERR_UNSUPPORTED;
    const int eb = dtype == TSLT_F32 ? 4 : 2;
    if (B < 0 || gamma < 0 || V <= 0 || k <= 0 || k > V || !(top_p > 0.0f) || !(temperature > 0.0f) ||
        !isfinite(temperature) || num_samples < 0)
        return TSLT_ERR_INVALID_ARG;
    if (k > TSLT_MAX_K) return TSLT_ERR_UNSUPPORTED;
    const long long rows_ll = (long long)B * gamma;
    if (rows_ll > 0x7fffffffLL / 64) return TSLT_ERR_UNSUPPORTED;
    if ((long long)V * eb > (1LL << 30)) return TSLT_ERR_UNSUPPORTED;  // tile and vector numbers stay well inside 32 bits
    const int rows = (int)rows_ll;
    if (rows == 0) return TSLT_OK;
    if (!logits || !idx || !logit || !count || !workspace || (num_samples > 0 && (!uniforms || !token)))
        return TSLT_ERR_INVALID_ARG;
    if (row_stride_elems < V || ((uintptr_t)logits & 15) || ((row_stride_elems * eb) & 15) ||
        ((uintptr_t)workspace & 255))
        return TSLT_ERR_INVALID_ARG;
    SparsifyPlan pl = make_sparsify_plan(rows, V, k, eb);
    if (workspace_bytes < pl.ws_bytes) return TSLT_ERR_WORKSPACE;

    SparsifyParams p;
    p.logits = (const unsigned char*)logits;
    p.row_stride_bytes = row_stride_elems * eb;
    p.V = V; p.rows = rows; p.k = k;
    p.top_p = top_p;
    p.c = make_scale(temperature);
    p.num_samples = num_samples;
    p.uniforms = uniforms;
    p.idx = idx; p.logit = logit; p.count = count; p.token = token; p.lse = lse; p.mass = mass;
    p.nchunks = pl.nchunks; p.split = pl.split;
    p.group_log2 = pl.group_log2; p.ngroups = pl.ngroups; p.tile_cap = pl.tile_cap;
    p.poll_limit = g_sparsify_poll_limit;
    unsigned char* ws = (unsigned char*)workspace;
    p.status = (int*)ws;
    p.seg_ready = (int*)(ws + pl.ws_ready_off);
    p.seg_stats = (SegStat*)(ws + pl.ws_stats_off);
    p.tile_max = (unsigned short*)(ws + pl.ws_tiles_off);

    cudaStream_t st = (cudaStream_t)stream;
    if (dtype == TSLT_F32) sparsify_stream_kernel<float><<<pl.split.grid, kBlockThreads, 0, st>>>(p);
    else sparsify_stream_kernel<bf16_t><<<pl.split.grid, kBlockThreads, 0, st>>>(p);
    if (cudaGetLastError() != cudaSuccess) return TSLT_ERR_CUDA;
    auto fin = dtype == TSLT_F32 ? sparsify_finish_kernel<float> : sparsify_finish_kernel<bf16_t>;
    static_assert(kFinishHeaderBytes + kSelBins * 4 + kMaxGroups * 4 + TSLT_MAX_K * 16 + TSLT_MAX_K * 8 <= 48 * 1024,
                  "the finish kernel's shared memory stays under the default limit");
    if (launch_dependent(fin, rows, kFinishThreads, pl.fin_smem, st, p) != cudaSuccess) return TSLT_ERR_CUDA;
    return TSLT_OK;
}
