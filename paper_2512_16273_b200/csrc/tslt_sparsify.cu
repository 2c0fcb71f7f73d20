// tslt_sparsify: draft-side sparsify-then-sample (Section 3, Solution 1; the sampling steps
// of Algorithms 2 and 4) as two kernels on the caller's stream.
//
// Streaming kernel.  One CTA reads one segment of one logits row from HBM exactly once, with
// 16-byte loads that go straight to registers (each warp instruction covers 512 contiguous
// bytes; two 2 KB chunks per warp are in flight).  It keeps two things: each lane's online
// (max, sum) for the softmax normaliser, and, for every 64-byte tile of the row (32 bf16 or 16 fp32
// logits), the top 16 bits of the tile's largest logit.  Nothing in the loop depends on k or top_p:
// no threshold, no histogram, no barrier, so it runs at the speed of a plain streaming reduction.
//   - Batches that fill the machine: one CTA per row.  The tile maxima stay in shared memory and, at
//     the end of the row, the CTA itself takes the tiles in groups so that there are two to four
//     times k groups, finds the k-th largest group maximum (a lower bound on the k-th largest logit:
//     each of the k groups at or above it holds a logit at or above it) and lists the tiles at or
//     above that bound in address order ("survivors": about 1.2 k of them).  Only the list goes to
//     the workspace.
//   - Smaller batches: rows are cut into segments so that every CTA slot has work; the tile maxima
//     go to the workspace (2 bytes per 64 read) and the finish kernel, which sees the whole row,
//     finds the bound and the survivors.
//
// Finish kernel (launched with programmatic stream serialization; a CTA starts on its row as soon
// as the row's segments have been handed over).  One CTA of 128 or 256 threads per row:
//   1. the survivors are read back from global memory: 64 bytes each, some k * 64 bytes of the
//      row's V * e;
//   2. their logits at or above the bound (the candidates, a little more than k) go to shared memory
//      in index order, by prefix sums over the survivors;
//   3. the exact k-th largest among them: by counting ranks while they are few, else by a two-pass
//      256-bin radix select on the 16-bit key (fp32 rows: once more on the low 16 bits); ties at the
//      k-th logit go to the lower index; the winners are compacted in place and so come out in
//      ascending token index without any sort;
//   4. the top-rho cut (a bitwise descent on the crossing key over fixed-point masses, no sort), the
//      renormalised distribution and its CDF in fp64, the samples by inverse CDF, the outputs.
// A row whose survivors or candidates do not fit their lists (thousands of tied maxima: constant
// rows, rows sorted by value; k close to V) runs the selection over the survivors' vectors, or all
// of the row's, in global memory instead: a histogram select and two more passes, slower, exact.
//
// Vocabulary shards: tslt_sparsify_shard is the same pair of kernels on a slice of the vocabulary;
// sparsify_merge_kernel joins the shards' lists with steps 3 and 4 of the finish kernel.
#include <math.h>

#include "tslt_common.cuh"
#include "tslt_rowmath.cuh"

namespace tslt {

constexpr int kTilesPerChunk = 32;        // 64-byte tiles in a 2 KB chunk
constexpr int kVecsPerTile = 4;           // 16-byte vectors in a tile
constexpr int kSparsifyStreamCtasPerSm = 4;  // 64 registers: two chunks per warp in flight (5 CTAs with one chunk in flight: 1.5 % slower; 3 CTAs: 4 % slower)
constexpr int kMaxGroups = 4096;          // group maxima the finish kernel bisects over
constexpr int kMaxTileList = 4096;        // survivor tiles it can list
constexpr int kSelBins = 1024;            // bins of the selection histogram
constexpr int kMaxShards = TSLT_MAX_SHARDS;  // vocabulary shards one merge takes
constexpr int kMaxMergeList = 2048;       // candidates the merge holds (nshards * k)
constexpr int kListPerThread = 8;         // candidate list entries per thread of a finishing CTA: lists of at most 8 * NT
constexpr int kWinnersPerThread = 4;      // winners per thread in the top-rho cut: k <= 4 * NT
constexpr uint32_t kLowestFinite16 = 0x0080u;   // key of -FLT_MAX >> 16
constexpr uint32_t kHighestFinite16 = 0xff7fu;  // key of +FLT_MAX >> 16

// What a segment hands over besides its tile maxima or its survivor list: one (max, sum) pair per
// warp and, from a segment that is a whole row, the outcome of its own selection.
struct SegStat {
    double S[kWarps];  // sum of 2^(y - M) over the warp's chunks of the segment
    float M[kWarps];   // the warp's reference exponent (base 2)
    int n_list;        // survivor tiles listed (-1: they did not fit the list)
    int bound16;       // 16-bit key at or below the row's k-th largest logit's (0: none)
    int max16;         // 16-bit key of the row's largest tile maximum
    int pad[5];
};
static_assert(sizeof(SegStat) == 128, "one record per 128 bytes");

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
    double* lse2;     // optional: the row's base-2 log-normaliser in fp64 (what a vocabulary shard hands to the merge)
    int nchunks;
    RowSplit split;
    int group_log2;   // tiles per group = 1 << group_log2
    int ngroups;      // <= kMaxGroups
    int tile_cap;     // survivor list capacity (<= kMaxTileList)
    int cand_cap;     // candidate list capacity (<= 8 * the finish kernel's threads)
    int poll_limit;   // polls of a segment's ready flag before falling back to the end of the streaming kernel
    int* status;
    int* seg_ready;           // [rows * nseg]
    SegStat* seg_stats;       // [rows * nseg]
    unsigned short* tile_max; // rows cut into segments: [rows, nchunks * 32], top 16 bits of each tile's largest logit, slot order
    uint32_t* row_list;       // whole-row CTAs: [rows, tile_cap] survivor tiles in address order
    int local_bound;          // 1: each row is one streaming CTA, which finds the bound and lists the survivors itself
    // merge of vocabulary shards only: what the shards handed over, [nshards, rows, part_k] / [nshards, rows]
    int nshards, part_k;
    const int* part_idx;
    const float* part_logit;
    const int* part_count;
    const double* part_lse2;
    int shard_offset[kMaxShards];  // token index of each shard's first logit
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

// Atomics on shared memory through the shared-space address: a generic-address atomic that happens to
// hit shared memory is several times slower, and the compiler cannot always tell.
__device__ __forceinline__ void smem_add(void* p, uint32_t v) {
    asm volatile("red.shared.add.u32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}
__device__ __forceinline__ void smem_add64(void* p, unsigned long long v) {
    asm volatile("red.shared.add.u64 [%0], %1;" ::"r"(smem_u32(p)), "l"(v) : "memory");
}
__device__ __forceinline__ void smem_max(void* p, uint32_t v) {
    asm volatile("red.shared.max.u32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}
__device__ __forceinline__ void smem_min(void* p, uint32_t v) {
    asm volatile("red.shared.min.u32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}

template <int NT> __device__ __forceinline__ void fsync() { asm volatile("bar.sync 1, %0;" ::"n"(NT) : "memory"); }

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

// Exclusive prefix sum of one int per thread over the NT threads; *total gets the sum.
template <int NT> __device__ __forceinline__ int block_exscan(int v, int tid, int* scr /* >= NT / 32 */, int* total) {
    const int lane = tid & 31, warp = tid >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) scr[warp] = incl;
    fsync<NT>();
    int base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) {
        const int t = scr[w];
        if (w < warp) base += t;
        tot += t;
    }
    fsync<NT>();
    *total = tot;
    return base + incl - v;
}
template <int NT> __device__ __forceinline__ double block_max_f64(double v, int tid, double* scr) {
    v = warp_max(v);
    if ((tid & 31) == 0) scr[tid >> 5] = v;
    fsync<NT>();
    double m = scr[0];
#pragma unroll
    for (int w = 1; w < NT / 32; ++w) m = fmax(m, scr[w]);
    fsync<NT>();
    return m;
}
template <int NT> __device__ __forceinline__ double block_sum_f64(double v, int tid, double* scr) {
    v = warp_sum(v);
    if ((tid & 31) == 0) scr[tid >> 5] = v;
    fsync<NT>();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) t += scr[w];
    fsync<NT>();
    return t;
}
// In-place inclusive scan of a[0..n) (shared memory, fp64).  Each thread owns a contiguous run, so
// the sums have a fixed order: deterministic.
template <int NT> __device__ __forceinline__ void block_inclusive_scan_f64(double* a, int n, int tid, double* scr) {
    const int per = (n + NT - 1) / NT;
    const int lo = min(n, tid * per), hi = min(n, lo + per);
    double run = 0.0;
    for (int i = lo; i < hi; ++i) run += a[i];
    double incl = run;
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) scr[warp] = incl;
    fsync<NT>();
    double base = 0.0;
    for (int w = 0; w < warp; ++w) base += scr[w];
    double acc = base + (incl - run);
    for (int i = lo; i < hi; ++i) {
        acc += a[i];
        a[i] = acc;
    }
    fsync<NT>();
}
// The kk-th largest of the thread block's 16-bit values (at least kk of them exist), by two histogram
// passes of 256 bins: the high byte, then the low byte among the values that share it.  A bisection
// on the value's bits would take one barrier per bit, and the keys of logits that straddle zero
// differ in nearly all sixteen.  for_each(f) calls f(v) for every value v of THIS thread.  *above
// gets the number of values larger than the result.  hist: 256 words of shared memory.  Ends with
// a barrier after the last read of sel, so both can be reused right away.
template <int NT, typename ForEach>
__device__ __forceinline__ uint32_t radix_kth16(int kk, ForEach for_each, uint32_t* hist, int* sel /* 2 words of shared memory */, int tid, int* above) {
    uint32_t prefix = 0;
    int above_acc = 0;
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {
        for (int i = tid; i < 256; i += NT) hist[i] = 0u;
        fsync<NT>();
        if (pass == 0) for_each([&](uint32_t v) { smem_add(&hist[v >> 8], 1u); });
        else for_each([&](uint32_t v) { if ((v >> 8) == prefix) smem_add(&hist[v & 255u], 1u); });
        fsync<NT>();
        if (tid < 32) {
            // rows of 32 bins from the top; lane l takes bin top - l of the row
            uint32_t carried = 0;
            int found_bin = 0;
            uint32_t found_above = 0;
            bool found = false;
            for (int top = 255; top >= 0; top -= 32) {
                const uint32_t cnt = hist[top - tid];
                uint32_t incl = cnt;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
                    if (tid >= o) incl += t;
                }
                const unsigned hit = __ballot_sync(0xffffffffu, carried + incl >= (uint32_t)kk);
                if (hit) {
                    const int l = __ffs(hit) - 1;
                    found_bin = top - l;
                    found_above = carried + __shfl_sync(0xffffffffu, incl - cnt, l);
                    found = true;
                    break;
                }
                carried += __shfl_sync(0xffffffffu, incl, 31);
            }
            if (tid == 0) {
                sel[0] = found ? found_bin : 0;
                sel[1] = found ? (int)found_above : 0;
            }
        }
        fsync<NT>();
        const int bin = sel[0], ab = sel[1];
        above_acc += ab;
        kk -= ab;
        prefix = pass == 0 ? (uint32_t)bin : ((prefix << 8) | (uint32_t)bin);
        fsync<NT>();
    }
    *above = above_acc;
    return prefix;
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

// Group maxima of one 64-byte line of tile maxima (32 slots, two per word): the packed bf16 maximum
// works on the raw top-16-bit patterns whatever the logits' type.  Writes the line's 32 >> glog group
// maxima (as keys) to gm_line, for 0 <= glog <= 5; returns the line's maximum as a raw pattern.
__device__ __forceinline__ uint32_t half_max(uint32_t w) { return bf16x2_max(w, w >> 16) & 0xffffu; }
__device__ __forceinline__ uint32_t line_group_maxima(const uint32_t (&w)[16], int glog, uint32_t* gm_line) {
    uint32_t t8[8], t4[4], t2[2];
#pragma unroll
    for (int i = 0; i < 8; ++i) t8[i] = bf16x2_max(w[2 * i], w[2 * i + 1]);
#pragma unroll
    for (int i = 0; i < 4; ++i) t4[i] = bf16x2_max(t8[2 * i], t8[2 * i + 1]);
    t2[0] = bf16x2_max(t4[0], t4[1]);
    t2[1] = bf16x2_max(t4[2], t4[3]);
    const uint32_t t1 = bf16x2_max(t2[0], t2[1]);
    if (glog == 0) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            gm_line[2 * i] = raw16_to_key16(w[i] & 0xffffu);
            gm_line[2 * i + 1] = raw16_to_key16(w[i] >> 16);
        }
    } else if (glog == 1) {
#pragma unroll
        for (int i = 0; i < 16; ++i) gm_line[i] = raw16_to_key16(half_max(w[i]));
    } else if (glog == 2) {
#pragma unroll
        for (int i = 0; i < 8; ++i) gm_line[i] = raw16_to_key16(half_max(t8[i]));
    } else if (glog == 3) {
#pragma unroll
        for (int i = 0; i < 4; ++i) gm_line[i] = raw16_to_key16(half_max(t4[i]));
    } else if (glog == 4) {
        gm_line[0] = raw16_to_key16(half_max(t2[0]));
        gm_line[1] = raw16_to_key16(half_max(t2[1]));
    } else if (glog == 5) {
        gm_line[0] = raw16_to_key16(half_max(t1));
    }
    return half_max(t1);
}

// Which of a line's 32 tiles have a key >= bound: bit a of the result is tile a of the chunk in
// ADDRESS order (tile j * 8 + q sits in slot q * 4 + j of the line).
__device__ __forceinline__ uint32_t line_survivors(const uint32_t (&w)[16], uint32_t bound) {
    uint32_t m = 0;
    {   // most lines hold no survivor: their maximum settles it
        uint32_t t = bf16x2_max(bf16x2_max(bf16x2_max(w[0], w[1]), bf16x2_max(w[2], w[3])),
                                bf16x2_max(bf16x2_max(w[4], w[5]), bf16x2_max(w[6], w[7])));
        t = bf16x2_max(t, bf16x2_max(bf16x2_max(bf16x2_max(w[8], w[9]), bf16x2_max(w[10], w[11])),
                                     bf16x2_max(bf16x2_max(w[12], w[13]), bf16x2_max(w[14], w[15]))));
        if (raw16_to_key16(half_max(t)) < bound) return 0u;
    }
#pragma unroll
    for (int a = 0; a < kTilesPerChunk; ++a) {
        const int slot = ((a & 7) << 2) | (a >> 3);
        const uint32_t raw = (slot & 1) ? (w[slot >> 1] >> 16) : (w[slot >> 1] & 0xffffu);
        m |= (raw16_to_key16(raw) >= bound ? 1u : 0u) << a;
    }
    return m;
}
__device__ __forceinline__ void load_line(const unsigned short* line, uint32_t (&w)[16]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint4 v = __ldcg(reinterpret_cast<const uint4*>(line) + i);
        w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
    }
}

// Shared memory of a whole-row streaming CTA (kLocal): header | histogram (256 words) | the row's tile
// maxima (2 bytes per tile, slot order) | the group maxima (2 bytes per group).
struct StreamShared {
    int sel[2];
    int iscr[8];
    int gmax;
    int pad[5];
};
constexpr int kStreamHeaderBytes = 64 + 256 * 4;
constexpr int kWarpSelectMax = 512;  // group maxima up to which one warp selects the bound
__host__ __device__ inline size_t stream_smem_bytes(int nchunks, int ngroups) {
    return kStreamHeaderBytes + (size_t)nchunks * kTilesPerChunk * 2 + (((size_t)ngroups * 4 + 15) / 16) * 16;
}

// kLocal: the CTA streams a whole row, keeps the tile maxima in shared memory and, at the end of the
// row, finds the bound (the k-th largest group maximum) and lists the survivor tiles itself: the
// finish kernel then starts from the list, and no tile maximum ever goes to global memory.
// Otherwise (rows cut into segments, small batches) the tile maxima go to the workspace and the
// finish kernel, which sees the whole row, does that part.
template <typename T, bool kLocal>
__global__ void __launch_bounds__(kBlockThreads, kSparsifyStreamCtasPerSm) sparsify_stream_kernel(const SparsifyParams p) {
    extern __shared__ __align__(16) unsigned char stream_smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    TSLT_STAMP(blockIdx.x, 0);
    const RowWork wk = locate_work(p.split, blockIdx.x, p.nchunks);
    const unsigned char* rowp = p.logits + (long long)wk.row * p.row_stride_bytes;
    const RowExtent ext = row_extent<T>(p.V);
    const float c = p.c.f;
    const unsigned char* lane_rowp = rowp + lane * kVecBytes;
    int ch = wk.chunk_begin + warp;
    // two chunks per warp are in flight at any time (4 KB; 128 KB per SM with four CTAs): the loads of
    // chunk ch + 16 are issued as soon as chunk ch has been consumed
    LaneTile<T> lt, lt2;
    if (ch < wk.chunk_end) lt.load_lane(lane_rowp, ch * kVecsPerChunk, ext);  // in flight during the set-up below
    if (ch + kWarps < wk.chunk_end) lt2.load_lane(lane_rowp, (ch + kWarps) * kVecsPerChunk, ext);
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
    unsigned short* tmax = kLocal ? reinterpret_cast<unsigned short*>(stream_smem + kStreamHeaderBytes)
                                  : p.tile_max + (size_t)wk.row * p.nchunks * kTilesPerChunk;
    auto consume = [&](LaneTile<T>& t) {
        const float lm = t.reduce_max();
        const uint2 q = QuadMax<T>::keys(t);
        if ((lane & 3) == 0) *reinterpret_cast<uint2*>(tmax + ch * kTilesPerChunk + lane) = q;  // slots (lane >> 2) * 4 ..+3
        ls.raise_to(lm, c);
        t.accumulate(ls, c);
        if (ch + 2 * kWarps < wk.chunk_end) t.load_lane(lane_rowp, (ch + 2 * kWarps) * kVecsPerChunk, ext);
        ch += kWarps;
    };
    while (ch < wk.chunk_end) {
        consume(lt);
        if (ch < wk.chunk_end) consume(lt2);
    }
    TSLT_STAMP(blockIdx.x, 1);
    // hand-over: one (M, S) pair per warp
    const float Mw = warp_max(ls.M);
    const double Sw = warp_sum(ls.total_f64() * exp2((double)ls.M - (double)Mw));
    SegStat* st = &p.seg_stats[blockIdx.x];
    if (lane == 0) {
        st->S[warp] = Sw;
        st->M[warp] = Mw;
    }
    if (kLocal) {
        // ---- the row's bound and survivor list, from the tile maxima in shared memory -------------------
        StreamShared* sh = reinterpret_cast<StreamShared*>(stream_smem);
        uint32_t* hist = reinterpret_cast<uint32_t*>(stream_smem + 64);
        const int ntiles = p.nchunks * kTilesPerChunk;
        unsigned short* gm = tmax + ntiles;
        uint32_t* gmw = reinterpret_cast<uint32_t*>(gm);  // groups of several lines (glog > 5): few, kept as words
        const int glog = p.group_log2, ngroups = p.ngroups, k = p.k;
        if (tid == 0) sh->gmax = 0;
        if (glog > 5)
            for (int i = tid; i < ngroups; i += kBlockThreads) gmw[i] = 0u;
        __syncthreads();  // every warp's tile maxima are in place
        // thread t takes lines t, t + 256, ...; a line (the 32 tile maxima of a chunk, 64 bytes) is read
        // with four 16-byte loads and worked on in registers.  Rows of up to 256 chunks (512 KB) keep
        // their one line per thread in registers from here to the listing.
        uint32_t mx = 0;
        uint32_t w0[16];
        const bool one_line = p.nchunks <= kBlockThreads;
#pragma unroll
        for (int i = 0; i < 16; ++i) w0[i] = 0xff80ff80u;  // -inf: never a survivor
        for (int cl = tid; cl < p.nchunks; cl += kBlockThreads) {
            uint32_t w[16];
            const uint4* line = reinterpret_cast<const uint4*>(tmax + cl * kTilesPerChunk);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 v = line[i];
                w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
            }
            uint32_t gl[32];  // (only the first 32 >> glog are written, and only for glog <= 5)
            const uint32_t lm = raw16_to_key16(line_group_maxima(w, glog, gl));
            if (glog <= 5) {
                for (int i = 0; i < (kTilesPerChunk >> glog); ++i) gm[((cl * kTilesPerChunk) >> glog) + i] = (unsigned short)gl[i];
            } else {
                smem_max(&gmw[cl >> (glog - 5)], lm);  // groups of several lines: 32-bit words, see below
            }
            mx = max(mx, lm);
            if (one_line) {
#pragma unroll
                for (int i = 0; i < 16; ++i) w0[i] = w[i];
            }
        }
        mx = __reduce_max_sync(0xffffffffu, mx);
        if (lane == 0) smem_max(&sh->gmax, mx);
        __syncthreads();
        uint32_t bound = 0;
        if (ngroups >= k && ngroups <= kWarpSelectMax) {
            // few groups: one warp bisects on the 16 bits of the key, its values in registers, with no
            // block barrier per step (a barrier costs this CTA a good part of a microsecond while
            // four other CTAs stream on the SM); the others wait at the barrier below
            if (warp == 0) {
                uint32_t v[kWarpSelectMax / 32];
#pragma unroll
                for (int j = 0; j < kWarpSelectMax / 32; ++j) {
                    const int i = lane + 32 * j;
                    v[j] = i < ngroups ? (glog <= 5 ? (uint32_t)gm[i] : gmw[i]) : 0u;
                }
                uint32_t b = 0;
                for (int bit = 15; bit >= 0; --bit) {
                    const uint32_t cand = b | (1u << bit);
                    int cnt = 0;
#pragma unroll
                    for (int j = 0; j < kWarpSelectMax / 32; ++j) cnt += v[j] >= cand ? 1 : 0;
                    if (__reduce_add_sync(0xffffffffu, cnt) >= k) b = cand;
                }
                if (lane == 0) sh->sel[0] = (int)b;
            }
            __syncthreads();
            bound = (uint32_t)sh->sel[0];
        } else if (ngroups >= k) {
            int unused;
            if (glog <= 5) {
                bound = radix_kth16<kBlockThreads>(k, [&](auto f) {
                    for (int i = tid; i < ngroups; i += kBlockThreads) f((uint32_t)gm[i]);
                }, hist, sh->sel, tid, &unused);
            } else {
                bound = radix_kth16<kBlockThreads>(k, [&](auto f) {
                    for (int i = tid; i < ngroups; i += kBlockThreads) f(gmw[i]);
                }, hist, sh->sel, tid, &unused);
            }
        }
        const uint32_t lo16 = max(bound, kLowestFinite16);
        // survivors in address order, positions by a prefix sum per round of 256 lines
        uint32_t* list = p.row_list + (size_t)wk.row * p.tile_cap;
        int base = 0;
        bool fits = true;
        for (int c0 = 0; c0 < p.nchunks; c0 += kBlockThreads) {
            const int cl = c0 + tid;
            uint32_t m = 0;
            if (one_line) {
                m = line_survivors(w0, lo16);
            } else if (cl < p.nchunks) {
                uint32_t w[16];
                const uint4* line = reinterpret_cast<const uint4*>(tmax + cl * kTilesPerChunk);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint4 v = line[i];
                    w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
                }
                m = line_survivors(w, lo16);
            }
            int round_total;
            int pos = base + block_exscan<kBlockThreads>(__popc(m), tid, sh->iscr, &round_total);
            if (base + round_total > p.tile_cap) fits = false;
            if (fits) {
                while (m) {
                    const int a = __ffs(m) - 1;
                    m &= m - 1;
                    list[pos++] = (uint32_t)(cl * kTilesPerChunk + a);
                }
            }
            base += round_total;
        }
        if (tid == 0) {
            st->n_list = fits ? base : -1;
            st->bound16 = (int)bound;
            st->max16 = sh->gmax;
        }
    }
    __syncthreads();  // every warp's part of the hand-over is written
    if (tid == 0) publish_row_ready(&p.seg_ready[blockIdx.x]);
    TSLT_STAMP(blockIdx.x, 2);
}

// ---- finish kernel ---------------------------------------------------------------------------------
// NT threads per row: 128 (k <= 128) or 256.  Finishing a row is a chain of dependent steps (trips
// to L2 / HBM, bisection rounds, prefix sums), and most finish CTAs of a large batch only find room
// on an SM once the streaming kernel's last wave drains, so what the finish costs is the chain's
// length times the number of waves left then: the chain is kept to three trips to memory (the
// hand-over, the survivors' vectors, the outputs).
__host__ __device__ inline size_t align16(size_t x) { return (x + 15) / 16 * 16; }
__host__ __device__ inline int pow2_at_least(int n) {
    int p = 1;
    while (p < n) p <<= 1;
    return p;
}
__host__ __device__ constexpr int finish_threads(int k) { return k <= 512 ? 128 : 256; }
__host__ __device__ constexpr int finish_resident(int nt) { return nt == 128 ? 8 : (nt == 256 ? 4 : 2); }
constexpr int kSegmentFinishThreads = 256;
constexpr int kFinishHeaderBytes = 512;
constexpr int kRankListMax = 160;  // candidates up to which the k-th is found by counting ranks (n * n / NT compares)

// Dynamic shared memory of the finish kernel:
//   header | histogram | region A | region B | region C | line maxima
//   histogram: the selection histogram of the all-vectors path; else the rank-counting keys, the
//              256 bins of the radix selects and of the top-rho mass descent
//   region A:  group maxima (rows cut into segments only)
//   region B:  survivor tile list, later the CDF (fp64)
//   region C:  candidates (raw logit bits, token index), compacted in place to the winners
struct FinishLayout {
    size_t hist, a, b, c, lines, total;
};
__host__ __device__ inline FinishLayout finish_layout(int ngroups, int tile_cap, int cand_cap, int k, int nchunks, bool local) {
    FinishLayout L;
    L.hist = kFinishHeaderBytes;
    L.a = L.hist + (size_t)kSelBins * 4;
    L.b = L.a + align16(local ? 0 : (size_t)ngroups * 4);
    const size_t tb = (size_t)tile_cap * 4, wb = (size_t)k * 8;
    L.c = L.b + align16(tb > wb ? tb : wb);
    L.lines = L.c + (size_t)cand_cap * 8;
    L.total = L.lines + (local ? 0 : align16((size_t)nchunks * 2));
    return L;
}

struct FinishShared {
    double scratch[16];
    double lrow;  // base-2 log of the row's softmax normaliser
    int iscr[16];
    int sel_bin, sel_above, sel_eq, sel_total;
    int ready, gmax;
};

// The vectors a thread works on: units [u0, u1) of the row's survivor tiles (tl: their tile numbers in
// address order, four vectors each), or of the whole row (tl == nullptr: unit = vector).  f(z, vi)
// is called for each of them in ascending order with the vector's logits (-inf beyond the row).
template <typename T, typename F>
__device__ __forceinline__ void for_my_vectors(const unsigned char* rowp, const RowExtent& ext, int V, const uint32_t* tl,
                                               int u0, int u1, F f) {
    constexpr int kPer = Elt<T>::kPerVec;
    constexpr int kInFlight = 2;  // (the tiles were asked of L2 first: more loads in flight only cost registers and code: 6 were 3 % slower at k = 1024)
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

// All-vectors path only.  The kk-th largest of the values value_of(z) in [lo, hi] over the thread
// block's vectors (values outside the range, or negative, do not take part), by a histogram of
// kSelBins bins over the range, narrowed once more if the range is wider than the histogram.
// Results in sh: sel_bin = the value, sel_above = how many are larger (inside [lo, hi]), sel_eq =
// how many equal it, sel_total = how many lie in [lo, hi].  If fewer than kk lie in the range,
// sel_bin = -1 and only sel_total is meaningful.  All threads call it.
template <typename T, int NT, typename VF>
__device__ __forceinline__ void hist_select(const unsigned char* rowp, const RowExtent& ext, int V, const uint32_t* tl, int u0,
                                            int u1, VF value_of, int lo, int hi, int kk, FinishShared* sh, uint32_t* hist,
                                            int tid) {
    constexpr int kPer = Elt<T>::kPerVec;
    int above_acc = 0, total_first = -1;
    for (;;) {
        int s = 0;
        while (((hi - lo) >> s) >= kSelBins) ++s;
        for (int i = tid; i < kSelBins; i += NT) hist[i] = 0u;
        fsync<NT>();
        for_my_vectors<T>(rowp, ext, V, tl, u0, u1, [&](const float(&z)[kPer], int) {
            int cur = -1;
            uint32_t run = 0;
#pragma unroll
            for (int e = 0; e < kPer; ++e) {
                const int v = value_of(z[e]);
                if (v >= lo && v <= hi) {
                    const int b = (v - lo) >> s;
                    if (b != cur) {  // equal neighbours (ties) cost one atomic, not one each
                        if (run) smem_add(&hist[cur], run);
                        cur = b;
                        run = 0;
                    }
                    ++run;
                }
            }
            if (run) smem_add(&hist[cur], run);
        });
        fsync<NT>();
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
        fsync<NT>();
        const int bin = sh->sel_bin, above = sh->sel_above, eq = sh->sel_eq, total = sh->sel_total;
        fsync<NT>();
        if (total_first < 0) total_first = total;
        if (bin < 0 || s == 0) {
            if (tid == 0) {
                sh->sel_bin = bin < 0 ? -1 : lo + bin;
                sh->sel_above = above_acc + above;
                sh->sel_eq = eq;
                sh->sel_total = total_first;
            }
            fsync<NT>();
            return;
        }
        above_acc += above;
        kk -= above;
        lo = lo + (bin << s);
        hi = min(hi, lo + (1 << s) - 1);
    }
}

// 16-bit key of a finite logit (its order-preserving key's top half), -1 otherwise.
__device__ __forceinline__ int finite_key16(float z) {
    const uint32_t k16 = float_to_key(z) >> 16;
    return (k16 >= kLowestFinite16 && k16 <= kHighestFinite16) ? (int)k16 : -1;
}

// The exact top-k of a candidate list held in shared memory in ascending token index (c_raw: raw
// logit bits, c_idx: token indices, n_c <= 8 * NT entries): ties at the k-th logit go to the lower
// index.  The winners are compacted in place, still in ascending index; returns how many there are.
// All NT threads call it; hist holds kSelBins words (it doubles as the rank-counting keys).
template <typename T, int NT>
__device__ __forceinline__ int select_in_list(int k, uint32_t* c_raw, int* c_idx, int n_c, uint32_t* hist, FinishShared* sh, int tid) {
    constexpr bool kBf16 = (Elt<T>::kBytes == 2);
    constexpr int kHeld = kListPerThread;  // most list entries a thread owns (the host sees to it: lists of at most 8 * NT)
    unsigned long long* rkeys = reinterpret_cast<unsigned long long*>(hist);
    int n = 0;
    {
        // the candidates sit in shared memory in index order; thread t owns entries [i0, i1)
        const int ipt = (n_c + NT - 1) / NT;  // <= kHeld
        const int i0 = min(n_c, tid * ipt), i1 = min(n_c, i0 + ipt);
        uint32_t winmask = 0;  // bit j: entry i0 + j is a winner
        if (n_c <= k) {
            winmask = (i1 - i0) >= 32 ? 0xffffffffu : ((1u << (i1 - i0)) - 1u);
        } else if (n_c <= kRankListMax) {
            // few candidates: count each one's rank under (logit descending, index ascending)
            for (int i = tid; i < n_c; i += NT)
                rkeys[i] = ((unsigned long long)float_to_key(__uint_as_float(c_raw[i])) << 32) |
                           (unsigned long long)(0xffffffffu - (uint32_t)c_idx[i]);
            fsync<NT>();
            for (int i = i0; i < i1; ++i) {
                const unsigned long long mine = rkeys[i];
                int r = 0;
                for (int j = 0; j < n_c; ++j) r += rkeys[j] > mine ? 1 : 0;
                if (r < k) winmask |= 1u << (i - i0);
            }
        } else {
            // many candidates: the k-th largest 16-bit key by two histogram passes, (fp32 rows) the low
            // 16 bits inside that key the same way; ties by position
            int above = 0;
            const uint32_t e16 = radix_kth16<NT>(k, [&](auto f) {
                for (int i = i0; i < i1; ++i) f(float_to_key(__uint_as_float(c_raw[i])) >> 16);
            }, hist, &sh->sel_bin, tid, &above);
            int need = k - above;
            uint32_t e32;
            if (kBf16) {
                e32 = (e16 << 16) | ((e16 & 0x8000u) ? 0u : 0xffffu);  // keys of bf16 values: the low half follows the sign
            } else {
                int above2 = 0;
                const uint32_t low = radix_kth16<NT>(need, [&](auto f) {
                    for (int i = i0; i < i1; ++i) {
                        const uint32_t kz = float_to_key(__uint_as_float(c_raw[i]));
                        if ((kz >> 16) == e16) f(kz & 0xffffu);
                    }
                }, hist, &sh->sel_bin, tid, &above2);
                e32 = (e16 << 16) | low;
                need -= above2;
            }
            int c_eq = 0;
            for (int i = i0; i < i1; ++i) c_eq += float_to_key(__uint_as_float(c_raw[i])) == e32 ? 1 : 0;
            int tot_eq;
            const int eq_before = block_exscan<NT>(c_eq, tid, sh->iscr, &tot_eq);
            int ties_left = max(0, min(c_eq, need - eq_before));
            for (int i = i0; i < i1; ++i) {
                const uint32_t kz = float_to_key(__uint_as_float(c_raw[i]));
                bool win = kz > e32;
                if (kz == e32 && ties_left > 0) {
                    win = true;
                    --ties_left;
                }
                if (win) winmask |= 1u << (i - i0);
            }
        }
        // compact the winners in place: every thread reads its own first, then all write
        uint32_t my_raw[kHeld];
        int my_idx[kHeld];
        int my_wins = 0;
#pragma unroll
        for (int j = 0; j < kHeld; ++j)
            if ((winmask >> j) & 1u) {
                my_raw[my_wins] = c_raw[i0 + j];
                my_idx[my_wins] = c_idx[i0 + j];
                ++my_wins;
            }
        int wpos = block_exscan<NT>(my_wins, tid, sh->iscr, &n);
#pragma unroll
        for (int j = 0; j < kHeld; ++j)
            if (j < my_wins) {
                c_raw[wpos + j] = my_raw[j];
                c_idx[wpos + j] = my_idx[j];
            }
        fsync<NT>();
    }
    return n;
}

// Steps 6 and 7 of the finish: the top-rho cut of the n winners (c_raw / c_idx, ascending index), the
// renormalised truncated distribution and its CDF in fp64 (cum: >= k doubles), the samples by inverse
// CDF and the row's outputs.  L2 is the base-2 log of the full-vocabulary normaliser.  All NT threads call it.
template <typename T, int NT>
__device__ __forceinline__ void cut_sample_write(const SparsifyParams& p, int row, int n, uint32_t* c_raw, int* c_idx,
                                                 double L2, uint32_t* hist, double* cum, FinishShared* sh, int tid) {
    constexpr bool kBf16 = (Elt<T>::kBytes == 2);
    constexpr int kMine = kWinnersPerThread;  // most winners a thread owns in the top-rho cut (k <= 4 * NT, host-checked)
    const int lane = tid & 31, k = p.k;
    const int n0 = n;
    uint32_t* win_raw = c_raw;
    int* win_idx = c_idx;
    const double cf = (double)p.c.f;  // the scale the streaming sum used: keeps q consistent with the normaliser
    const double cd = p.c.d;
    double mass = 0.0;
    // ---- 6. top-rho cut ---------------------------------------------------------------------------------------
    // The smallest n whose cumulative q, in the order (logit descending, index ascending), reaches
    // top_p.  No sort: the key of the entry at which the cumulative crosses is the largest t with
    // mass(key >= t) >= top_p, found bit by bit with one block reduction per bit; then the ties of
    // that key, which all carry the same q, are counted off in index order.  Masses are summed as
    // 2^-62 fixed point, so the sums do not depend on the order of the adds: deterministic.  (A
    // histogram of mass per key byte needs 64-bit shared atomics on a handful of hot bins and was
    // three times slower than the sort it replaced; the bisection is three times faster.)
    if (n0 > 0 && p.top_p < 1.0f) {
        constexpr double kFix = 4611686018427387904.0;  // 2^62
        unsigned long long* mhist = reinterpret_cast<unsigned long long*>(hist);  // 256 bins
        const int ipt = (n0 + NT - 1) / NT;  // <= kMine
        const int i0 = min(n0, tid * ipt), i1 = min(n0, i0 + ipt);
        uint32_t kz[kMine];
        unsigned long long qf[kMine];
#pragma unroll
        for (int j = 0; j < kMine; ++j) {
            kz[j] = 0u;
            qf[j] = 0ull;
            if (i0 + j < i1) {
                const float z = __uint_as_float(win_raw[i0 + j]);
                kz[j] = float_to_key(z);
                qf[j] = __double2ull_rn(fmin(exp2((double)z * cf - L2), 1.0) * kFix);
            }
        }
        const unsigned long long target = __double2ull_rn((double)p.top_p * kFix);
        // mass of the entries whose key is >= t, over the block (fixed point: any order gives the same sum)
        auto mass_from = [&](uint32_t t, int slot) -> unsigned long long {
            unsigned long long m = 0ull;
#pragma unroll
            for (int j = 0; j < kMine; ++j)
                if (i0 + j < i1 && kz[j] >= t) m += qf[j];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m += __shfl_xor_sync(0xffffffffu, m, o);
            if (lane == 0 && m) smem_add64(&mhist[slot], m);  // one add per warp: 4 or 8 in all
            fsync<NT>();
            return mhist[slot];
        };
        for (int i = tid; i < 40; i += NT) mhist[i] = 0ull;
        if (tid == 0) sh->scratch[1] = 0.0;
        fsync<NT>();
        unsigned long long mass_above = 0ull;
        uint32_t prefix = 0u;
        bool crossed = mass_from(0u, 0) >= target;
        if (!crossed) {
            mass_above = mhist[0];  // the whole mass: the cumulative never reaches top_p, everything is kept
        } else {
            // the crossing key: the largest t with mass(key >= t) >= top_p, bit by bit
            int slot = 1;
            unsigned long long last_rejected = 0ull;
#pragma unroll 1
            for (int bit = 31; bit >= (kBf16 ? 16 : 0); --bit) {
                const uint32_t cand = prefix | (1u << bit);
                const unsigned long long m = mass_from(cand, slot++);
                if (m >= target) prefix = cand;
                else last_rejected = m;
            }
            mass_above = last_rejected;  // mass of the keys above the crossing key (the last candidate refused is that key + 1 ulp)
        }
        if (!crossed) {
            mass = (double)mass_above / kFix;
        } else {
            // (keys of bf16 values: the low half follows the sign and was not searched)
            const uint32_t ckey = kBf16 ? ((prefix & 0xffff0000u) | ((prefix & 0x80000000u) ? 0u : 0xffffu)) : prefix;
            // the ties of the crossing key share one q: how many of them, in index order, it takes
            int c_gt = 0, c_eq = 0;
            unsigned long long qk = 0ull;
#pragma unroll
            for (int j = 0; j < kMine; ++j)
                if (i0 + j < i1) {
                    c_gt += kz[j] > ckey ? 1 : 0;
                    if (kz[j] == ckey) {
                        ++c_eq;
                        qk = qf[j];
                    }
                }
            if (qk) sh->scratch[1] = __longlong_as_double((long long)qk);  // (every writer writes the same value)
            int tot_eq, tot_keep;
            const int eq_before = block_exscan<NT>(c_eq, tid, sh->iscr, &tot_eq);
            qk = (unsigned long long)__double_as_longlong(sh->scratch[1]);
            const unsigned long long missing = target - mass_above;  // > 0: the bins above did not reach it
            int need = qk ? (int)min((unsigned long long)tot_eq, (missing + qk - 1ull) / qk) : tot_eq;
            if (need < 1) need = 1;
            const int my_ties = max(0, min(c_eq, need - eq_before));
            // keep the larger keys and the first `need` ties: read mine, then (after the scan's barriers) write
            uint32_t keep_raw[kMine];
            int keep_idx[kMine];
            int kept = 0, ties_left = my_ties;
#pragma unroll
            for (int j = 0; j < kMine; ++j)
                if (i0 + j < i1) {
                    bool keep = kz[j] > ckey;
                    if (kz[j] == ckey && ties_left > 0) {
                        keep = true;
                        --ties_left;
                    }
                    if (keep) {
                        keep_raw[kept] = win_raw[i0 + j];
                        keep_idx[kept] = win_idx[i0 + j];
                        ++kept;
                    }
                }
            const int kp = block_exscan<NT>(kept, tid, sh->iscr, &tot_keep);
#pragma unroll
            for (int j = 0; j < kMine; ++j)
                if (j < kept) {
                    win_raw[kp + j] = keep_raw[j];
                    win_idx[kp + j] = keep_idx[j];
                }
            n = tot_keep;
            mass = (double)(mass_above + (unsigned long long)need * qk) / kFix;
            fsync<NT>();
        }
    }
    // ---- 7. renormalised truncated distribution in fp64, CDF, samples, outputs ----------------------------
    double my_max = -INFINITY;
    for (int i = tid; i < n; i += NT) my_max = fmax(my_max, (double)__uint_as_float(win_raw[i]) * cd);
    const double mS = block_max_f64<NT>(my_max, tid, sh->scratch);
    double my_mass = 0.0;
    for (int i = tid; i < n; i += NT) {
        const double z = (double)__uint_as_float(win_raw[i]);
        if (!(p.top_p < 1.0f)) my_mass += exp2(z * cf - L2);
        cum[i] = exp2(z * cd - mS);
    }
    if (!(p.top_p < 1.0f)) mass = block_sum_f64<NT>(my_mass, tid, sh->scratch);
    else fsync<NT>();
    block_inclusive_scan_f64<NT>(cum, n, tid, sh->scratch);

    int* o_idx = p.idx + (size_t)row * k;
    float* o_logit = p.logit + (size_t)row * k;
    for (int i = tid; i < k; i += NT) {
        o_idx[i] = i < n ? win_idx[i] : -1;
        o_logit[i] = i < n ? __uint_as_float(win_raw[i]) : -INFINITY;
    }
    if (tid == 0) {
        p.count[row] = n;
        if (p.lse) p.lse[row] = n0 > 0 ? (float)(L2 * 0.6931471805599453) : -INFINITY;
        if (p.mass) p.mass[row] = n0 > 0 ? (float)mass : 0.f;
        if (p.lse2) p.lse2[row] = n0 > 0 ? L2 : -INFINITY;
    }
    const double W = n > 0 ? cum[n - 1] : 0.0;
    for (int sidx = tid; sidx < p.num_samples; sidx += NT) {
        int tok = -1;
        if (n > 0) {
            const float u = clamp_uniform(p.uniforms[(size_t)row * p.num_samples + sidx]);
            int pos2 = first_greater(cum, n, (double)u * W);
            if (pos2 >= n) {
                pos2 = n - 1;
                while (pos2 > 0 && !(cum[pos2] - cum[pos2 - 1] > 0.0)) --pos2;  // the last entry with positive mass
            }
            tok = win_idx[pos2];
        }
        p.token[(size_t)row * p.num_samples + sidx] = tok;
    }
}

// Step 4 of the finish: the finite logits of the survivor tiles (tl: n_surv tile numbers in address
// order) at or above the bound go to the candidate list in shared memory, in ascending token index.
// Returns how many there are, or -1 if they do not fit cand_cap (nothing usable is written then).
template <typename T, int NT>
__device__ __forceinline__ int gather_candidates(const unsigned char* rowp, const RowExtent& ext, int V, const uint32_t* tl,
                                                 int n_surv, int lo16, int cand_cap, uint32_t* c_raw, int* c_idx,
                                                 FinishShared* sh, int tid) {
    constexpr int kPer = Elt<T>::kPerVec;
    // the vectors this thread works on: a contiguous run of the survivors' vectors, or of the row's
    const uint32_t* units = tl;
    const int n_units = tl ? n_surv * kVecsPerTile : (V + kPer - 1) / kPer;
    const int upt = (n_units + NT - 1) / NT;
    const int u0 = min(n_units, tid * upt), u1 = min(n_units, u0 + upt);
    const float lo_f = key_to_float((uint32_t)lo16 << 16);  // the smallest float whose 16-bit key is lo16
    auto is_candidate = [lo_f](float z) { return z >= lo_f && z <= 3.4028234e38f; };
    bool in_smem = false;
    int n_c = 0;
    {
        {
            // one pass over the thread's vectors; the first candidates it finds wait in a small
            // stash while the prefix sum finds where they go.  A thread that found more than its
            // stash holds reads its own vectors a second time (from L2).
            constexpr int kStash = 12;
            uint32_t st_raw[kStash];
            int st_idx[kStash];
            int cnt = 0;
            // every tile of this thread is asked of L2 first, so that the loads below (two vectors in
            // flight per thread) do not each pay a trip to HBM
            for (int u = u0; u < u1; ++u)
                if (u == u0 || (u & 3) == 0)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(rowp + (size_t)tl[u >> 2] * (kVecsPerTile * kVecBytes)));
            for_my_vectors<T>(rowp, ext, V, units, u0, u1, [&](const float(&z)[kPer], int vi) {
#pragma unroll
                for (int e = 0; e < kPer; ++e)
                    if (is_candidate(z[e])) {
                        if (cnt < kStash) {
                            st_raw[cnt] = __float_as_uint(z[e]);
                            st_idx[cnt] = vi * kPer + e;
                        }
                        ++cnt;
                    }
            });
            int cpos = block_exscan<NT>(cnt, tid, sh->iscr, &n_c);
            if (n_c <= cand_cap) {
                in_smem = true;
                if (cnt <= kStash) {
                    for (int j = 0; j < cnt; ++j) {
                        c_raw[cpos + j] = st_raw[j];
                        c_idx[cpos + j] = st_idx[j];
                    }
                } else {
                    // (this thread alone reads its vectors again; they are in L2 now)
                    for_my_vectors<T>(rowp, ext, V, units, u0, u1, [&](const float(&z)[kPer], int vi) {
#pragma unroll
                        for (int e = 0; e < kPer; ++e)
                            if (is_candidate(z[e])) {
                                c_raw[cpos] = __float_as_uint(z[e]);
                                c_idx[cpos] = vi * kPer + e;
                                ++cpos;
                            }
                    });
                }
                fsync<NT>();
            }
        }
    }
    return in_smem ? n_c : -1;
}

// The rare rows whose survivors or candidates do not fit their lists (thousands of tied tile maxima;
// k close to V): the same selection over the survivors' vectors (tl), or all of the row's (tl ==
// nullptr), in global memory: a histogram for the 16-bit key (fp32 rows: another for the low 16 bits), a
// count and a collecting pass.  The winners go to c_raw / c_idx in ascending index; returns how many.
// hist: kSelBins words.  Kept out of line: it is several times the code of the common path.
template <typename T, int NT>
__device__ __noinline__ int select_from_global(const unsigned char* rowp, const RowExtent ext, int V, const uint32_t* tl,
                                               int n_surv, int lo16, int max16, int k, uint32_t* c_raw, int* c_idx,
                                               uint32_t* hist, FinishShared* sh, int tid) {
    constexpr bool kBf16 = (Elt<T>::kBytes == 2);
    constexpr int kPer = Elt<T>::kPerVec;
    // the vectors this thread works on: a contiguous run of the survivors' vectors, or of the row's
    const uint32_t* units = tl;
    const int n_units = tl ? n_surv * kVecsPerTile : (V + kPer - 1) / kPer;
    const int upt = (n_units + NT - 1) / NT;
    const int u0 = min(n_units, tid * upt), u1 = min(n_units, u0 + upt);
    const float lo_f = key_to_float((uint32_t)lo16 << 16);  // the smallest float whose 16-bit key is lo16
    auto is_candidate = [lo_f](float z) { return z >= lo_f && z <= 3.4028234e38f; };
    int n = 0;
        // The survivors do not fit (thousands of tied tile maxima, or more candidates than the list
        // holds): the same selection over the survivors' vectors, or all of the row's, in global
        // memory: a histogram for the 16-bit key (fp32 rows: another for the low 16 bits), a count
        // and a collecting pass.
        auto key16_of = [](float z) -> int { return finite_key16(z); };
        hist_select<T, NT>(rowp, ext, V, units, u0, u1, key16_of, lo16, max16, k, sh, hist, tid);
        const int e16 = sh->sel_bin, above = sh->sel_above, total = sh->sel_total;
        fsync<NT>();
        uint32_t e32 = 0;   // key of the k-th largest logit (0: fewer than k finite logits, all of them win)
        int need_ties = 0;  // how many logits equal to it are winners (the lowest indices)
        if (e16 >= 0) {
            if (kBf16) {
                e32 = ((uint32_t)e16 << 16) | ((e16 & 0x8000) ? 0u : 0xffffu);
                need_ties = k - above;
            } else {
                const uint32_t hi_bits = (uint32_t)e16;
                auto low16_of = [hi_bits](float z) -> int {
                    const uint32_t kz = float_to_key(z);
                    return (kz >> 16) == hi_bits ? (int)(kz & 0xffffu) : -1;
                };
                hist_select<T, NT>(rowp, ext, V, units, u0, u1, low16_of, 0, 0xffff, k - above, sh, hist, tid);
                const int low = sh->sel_bin, above2 = sh->sel_above;
                fsync<NT>();
                e32 = (hi_bits << 16) | (uint32_t)low;
                need_ties = k - above - above2;
            }
        }
        if (total > 0) {
            int c_gt = 0, c_eq = 0;
            for_my_vectors<T>(rowp, ext, V, units, u0, u1, [&](const float(&z)[kPer], int) {
#pragma unroll
                for (int e = 0; e < kPer; ++e) {
                    if (!is_candidate(z[e])) continue;
                    const uint32_t kz = float_to_key(z[e]);
                    c_gt += kz > e32 ? 1 : 0;
                    c_eq += kz == e32 ? 1 : 0;
                }
            });
            int tot_eq, tot_w;
            const int eq_before = block_exscan<NT>(c_eq, tid, sh->iscr, &tot_eq);
            const int my_ties = max(0, min(c_eq, need_ties - eq_before));
            int wpos = block_exscan<NT>(c_gt + my_ties, tid, sh->iscr, &tot_w);
            int ties_left = my_ties;
            for_my_vectors<T>(rowp, ext, V, units, u0, u1, [&](const float(&z)[kPer], int vi) {
#pragma unroll
                for (int e = 0; e < kPer; ++e) {
                    if (!is_candidate(z[e])) continue;
                    const uint32_t kz = float_to_key(z[e]);
                    bool win = kz > e32;
                    if (kz == e32 && ties_left > 0) {
                        win = true;
                        --ties_left;
                    }
                    if (win && wpos < k) {
                        c_raw[wpos] = __float_as_uint(z[e]);
                        c_idx[wpos] = vi * kPer + e;
                        ++wpos;
                    }
                }
            });
            n = min(tot_w, k);
            fsync<NT>();
        }
    return n;
}

template <typename T, int NT, bool kLocal>
__global__ void __launch_bounds__(NT, finish_resident(NT)) sparsify_finish_kernel(const SparsifyParams p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    FinishShared* sh = reinterpret_cast<FinishShared*>(smem_raw);
    static_assert(sizeof(FinishShared) <= kFinishHeaderBytes, "header");
    const int k = p.k;
    const FinishLayout L = finish_layout(p.ngroups, p.tile_cap, p.cand_cap, k, p.nchunks, kLocal);
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem_raw + L.hist);
    uint32_t* gm = reinterpret_cast<uint32_t*>(smem_raw + L.a);
    uint32_t* tl = reinterpret_cast<uint32_t*>(smem_raw + L.b);
    double* cum = reinterpret_cast<double*>(tl);
    uint32_t* c_raw = reinterpret_cast<uint32_t*>(smem_raw + L.c);
    int* c_idx = reinterpret_cast<int*>(c_raw + p.cand_cap);
    unsigned short* lmax = reinterpret_cast<unsigned short*>(smem_raw + L.lines);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, row = blockIdx.x;
    const int nseg = p.split.nseg, nchunks = p.nchunks;
    const unsigned char* rowp = p.logits + (long long)row * p.row_stride_bytes;
    const RowExtent ext = row_extent<T>(p.V);
    TSLT_STAMP(row, 3);
    if (tid == 0 && p.num_samples > 0)  // the uniforms are needed last: ask for their cache line now
        asm volatile("prefetch.global.L2 [%0];" ::"l"(p.uniforms + (size_t)row * p.num_samples));
    if (tid == 0) sh->gmax = 0;
    const int glog = p.group_log2, ngroups = p.ngroups;
    if (glog > 5 && !kLocal)
        for (int i = tid; i < ngroups; i += NT) gm[i] = 0u;
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
    fsync<NT>();
    if (!sh->ready) {
        if (tid == 0) atomicOr(p.status, TSLT_STATUS_WAIT_FELL_BACK);
        wait_for_primary_kernel();
    }
    fsync<NT>();
    TSLT_STAMP(row, 4);
    // ---- the row's log-normaliser, by one warp (fp64 is scarce) -------------------------------------
    if (warp == 1) {
        // every (max, sum) pair is asked for before any is used: one trip to memory
        const SegStat* st = p.seg_stats + (size_t)row * nseg;
        constexpr int kPairs = 4;  // per lane and round: 128 pairs = 16 segments a round
        double Mall = -INFINITY, Sall = 0.0;
        for (int base = 0; base < nseg * kWarps; base += 32 * kPairs) {
            double Sw[kPairs], Mw[kPairs];
#pragma unroll
            for (int j = 0; j < kPairs; ++j) {
                const int i = base + j * 32 + lane;
                const bool in = i < nseg * kWarps;
                Sw[j] = in ? __ldcg(&st[i / kWarps].S[i % kWarps]) : 0.0;
                Mw[j] = in ? (double)__ldcg(&st[i / kWarps].M[i % kWarps]) : -INFINITY;
            }
            double Mnew = Mall;
#pragma unroll
            for (int j = 0; j < kPairs; ++j)
                if (Sw[j] > 0.0) Mnew = fmax(Mnew, Mw[j]);
            Mnew = warp_max(Mnew);
            double add = 0.0;
#pragma unroll
            for (int j = 0; j < kPairs; ++j)
                if (Sw[j] > 0.0) add += Sw[j] * exp2(Mw[j] - Mnew);
            Sall = (Sall > 0.0 ? Sall * exp2(Mall - Mnew) : 0.0) + warp_sum(add);
            Mall = Mnew;
        }
        if (lane == 0) sh->lrow = Sall > 0.0 ? Mall + log2(Sall) : -INFINITY;
    }
    int lo16, max16, n_surv;
    bool listed;
    if (kLocal) {
        // ---- 1-3 done by the row's streaming CTA: its bound, its survivor list ------------------------------
        const SegStat* st = p.seg_stats + row;
        const int n_list = __ldcg(&st->n_list);
        lo16 = max(__ldcg(&st->bound16), (int)kLowestFinite16);
        max16 = min(__ldcg(&st->max16), (int)kHighestFinite16);
        listed = n_list >= 0 && n_list <= p.tile_cap;
        n_surv = listed ? n_list : 0;
        const uint32_t* list = p.row_list + (size_t)row * p.tile_cap;
        for (int i = tid; i < n_surv; i += NT) tl[i] = __ldcg(list + i);
        fsync<NT>();
    } else {
        // ---- 1. group maxima of the tile maxima; each line's maximum is kept for step 3 -------------------
        // Thread t takes a run of consecutive chunks; a chunk's 32 tile maxima are one 64-byte line.
        const unsigned short* tmax = p.tile_max + (size_t)row * nchunks * kTilesPerChunk;
        const int cpt = (nchunks + NT - 1) / NT;
        const int ch0 = min(nchunks, tid * cpt), ch1 = min(nchunks, ch0 + cpt);
        // (keeping a thread's lines in registers from here to step 3 saved one trip to L2 and cost 32
        // registers across the whole finish: the chain was 4 us longer on the smallest batches)
        for (int ch = ch0; ch < ch1; ++ch) {
            uint32_t w[16];
            load_line(tmax + ch * kTilesPerChunk, w);
            const uint32_t lm = line_group_maxima(w, glog, gm + ((ch * kTilesPerChunk) >> (glog <= 5 ? glog : 5)));
            if (glog > 5) smem_max(&gm[ch >> (glog - 5)], raw16_to_key16(lm));
            lmax[ch] = (unsigned short)lm;
        }
        fsync<NT>();
        {
            uint32_t mx = 0u;
            for (int i = tid; i < ngroups; i += NT) mx = max(mx, gm[i]);
            mx = __reduce_max_sync(0xffffffffu, mx);
            if (lane == 0) smem_max(&sh->gmax, mx);
        }
        fsync<NT>();
        const uint32_t gmax = (uint32_t)sh->gmax;
        max16 = min((int)gmax, (int)kHighestFinite16);
        // ---- 2. the k-th largest group maximum: a lower bound on the k-th largest logit's key ---------------
        uint32_t bound = 0;
        if (ngroups >= k) {
            int unused;
            bound = radix_kth16<NT>(k, [&](auto f) {
                for (int i = tid; i < ngroups; i += NT) f(gm[i]);
            }, hist, &sh->sel_bin, tid, &unused);
        }
        lo16 = max((int)bound, (int)kLowestFinite16);
        // ---- 3. survivor tiles (key >= bound), listed in address order -----------------------------------------
        int my_surv = 0;
        for (int ch = ch0; ch < ch1; ++ch) {
            if (raw16_to_key16(lmax[ch]) < (uint32_t)lo16) continue;
            uint32_t w[16];
            load_line(tmax + ch * kTilesPerChunk, w);
            my_surv += __popc(line_survivors(w, (uint32_t)lo16));  // bit a: tile a of the chunk (none beyond the row)
        }
        int pos = block_exscan<NT>(my_surv, tid, sh->iscr, &n_surv);
        listed = n_surv <= p.tile_cap;
        if (listed) {
            for (int ch = ch0; ch < ch1; ++ch) {
                if (raw16_to_key16(lmax[ch]) < (uint32_t)lo16) continue;
                uint32_t w[16];
                load_line(tmax + ch * kTilesPerChunk, w);
                uint32_t m = line_survivors(w, (uint32_t)lo16);
                while (m) {
                    const int a = __ffs(m) - 1;
                    m &= m - 1;
                    tl[pos++] = (uint32_t)(ch * kTilesPerChunk + a);
                }
            }
        }
        fsync<NT>();
    }
    TSLT_STAMP(row, 5);
    const double L2 = sh->lrow;
    // ---- 4. candidates in shared memory, 5. the exact top-k (ties to the lower index), ascending index ----
    if (!listed) lo16 = (int)kLowestFinite16;
    int n = 0;
    if (max16 >= lo16) {
        const int n_c = listed ? gather_candidates<T, NT>(rowp, ext, p.V, tl, n_surv, lo16, p.cand_cap, c_raw, c_idx, sh, tid) : -1;
        TSLT_STAMP(row, 6);
        if (n_c >= 0) n = select_in_list<T, NT>(k, c_raw, c_idx, n_c, hist, sh, tid);
        else n = select_from_global<T, NT>(rowp, ext, p.V, listed ? tl : nullptr, n_surv, lo16, max16, k, c_raw, c_idx, hist, sh, tid);
    }
    TSLT_STAMP(row, 7);
    cut_sample_write<T, NT>(p, row, n, c_raw, c_idx, L2, hist, cum, sh, tid);
    TSLT_STAMP(row + kStampCtas / 2, 0);
    // this kernel's completion must imply the streaming kernel's (what follows on the stream relies
    // on it): one CTA sees to that; the others leave and make room
    if (row == 0) wait_for_primary_kernel();
}

// ---- merge of vocabulary shards ------------------------------------------------------------------------
// One CTA of 256 threads per row.  The shards' (index, logit) lists, each ascending in its own
// indices, laid end to end in shard order are one candidate list in ascending token index: exactly
// what the finish kernel's selection works on.  The row's normaliser is the sum of the shards'.
constexpr int kMergeThreads = 256;
template <typename T>
__global__ void __launch_bounds__(kMergeThreads, 4) sparsify_merge_kernel(const SparsifyParams p) {
    constexpr int NT = kMergeThreads;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    FinishShared* sh = reinterpret_cast<FinishShared*>(smem_raw);
    const int k = p.k;
    const FinishLayout L = finish_layout(0, 0, p.cand_cap, k, 0, true);
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem_raw + L.hist);
    double* cum = reinterpret_cast<double*>(smem_raw + L.b);
    uint32_t* c_raw = reinterpret_cast<uint32_t*>(smem_raw + L.c);
    int* c_idx = reinterpret_cast<int*>(c_raw + p.cand_cap);
    const int tid = threadIdx.x, lane = tid & 31, row = blockIdx.x, S = p.nshards;
    if (row == 0 && tid == 0) *p.status = 0;  // this call's first (and only) kernel
    if (tid < 32) {
        // where each shard's entries go, and the row's log-normaliser
        int cnt = 0;
        double l2 = -INFINITY;
        if (lane < S) {
            cnt = p.part_count[(size_t)lane * p.rows + row];
            cnt = cnt < 0 ? 0 : (cnt > p.part_k ? p.part_k : cnt);
            l2 = p.part_lse2[(size_t)lane * p.rows + row];
            if (!(l2 > -INFINITY) || !(l2 < INFINITY)) l2 = -INFINITY;  // an empty shard (or a NaN)
        }
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane < S) sh->iscr[lane] = incl - cnt;
        const double M = warp_max(l2);
        const double sum = warp_sum(l2 > -INFINITY ? exp2(l2 - M) : 0.0);
        if (lane == 31) sh->sel_total = incl;
        if (lane == 0) sh->lrow = sum > 0.0 ? M + log2(sum) : -INFINITY;
    }
    fsync<NT>();
    const int n_c = sh->sel_total;
    const double L2 = sh->lrow;
    for (int s = 0; s < S; ++s) {
        const int base = sh->iscr[s];
        const int cnt = (s + 1 < S ? sh->iscr[s + 1] : n_c) - base;
        const size_t src = ((size_t)s * p.rows + row) * p.part_k;
        for (int i = tid; i < cnt; i += NT) {
            c_raw[base + i] = __float_as_uint(p.part_logit[src + i]);
            c_idx[base + i] = p.part_idx[src + i] + p.shard_offset[s];
        }
    }
    fsync<NT>();
    const int n = select_in_list<T, NT>(k, c_raw, c_idx, n_c, hist, sh, tid);
    cut_sample_write<T, NT>(p, row, n, c_raw, c_idx, L2, hist, cum, sh, tid);
}

}  // namespace tslt

// ---- host side -------------------------------------------------------------------------------
namespace tslt {

struct SparsifyPlan {
    int nchunks, group_log2, ngroups, tile_cap, cand_cap, fin_threads;
    RowSplit split;
    bool local_bound;    // whole-row streaming CTAs find the bound and list the survivors themselves
    size_t stream_smem;  // their shared memory
    size_t fin_smem;
    size_t ws_ready_off, ws_stats_off, ws_tiles_off, ws_bytes;
};
constexpr size_t kStreamSmemLimit = 100 * 1024;

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
    pl.tile_cap = 2 * k < 512 ? 512 : (2 * k > kMaxTileList ? kMaxTileList : 2 * k);  // some 1.1 to 1.4 k survive
    pl.cand_cap = 2 * k < 512 ? 512 : (2 * k > 2048 ? 2048 : 2 * k);
    pl.fin_threads = finish_threads(k);
    pl.fin_smem = 0;  // (set below, once the split is known)
    // One CTA per row when the rows fill the machine; fewer rows are cut into segments (at least one
    // chunk per warp each) so that every CTA slot has work.  A segment costs nothing but its own
    // hand-over (8 (max, sum) pairs and a flag).
    const int slots = kSparsifyStreamCtasPerSm * sm_count_cached();
    // (Cutting the rows of a large batch as well, into segments of 64 to 256 KB, was measured and
    // dropped: the finish kernel is only scheduled once every streaming CTA has started, which with
    // eight times the CTAs is the very end of the streaming kernel.)
    int nseg = 1;
    if (rows > 0 && rows < slots) {
        nseg = slots / rows;  // (one wave: a CTA that had to wait for a slot would double the streaming time)
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
    pl.stream_smem = stream_smem_bytes(pl.nchunks, pl.ngroups);
    pl.local_bound = pl.split.nseg == 1 && pl.stream_smem <= kStreamSmemLimit;
    // rows cut into segments are few: a finish CTA has its SM to itself and the row's latency is what counts
    if (!pl.local_bound) pl.fin_threads = kSegmentFinishThreads;
    if (!pl.local_bound) pl.stream_smem = 0;
    pl.fin_smem = finish_layout(pl.ngroups, pl.tile_cap, pl.cand_cap, k, pl.nchunks, pl.local_bound).total;
    size_t off = kWsHeaderBytes;
    pl.ws_ready_off = off;
    off = align_up256(off + (size_t)rows * pl.split.nseg * sizeof(int));
    pl.ws_stats_off = off;
    off = align_up256(off + (size_t)rows * pl.split.nseg * sizeof(SegStat));
    pl.ws_tiles_off = off;
    // whole-row CTAs hand a survivor list over, segments their tile maxima
    off = align_up256(off + (pl.local_bound ? (size_t)rows * pl.tile_cap * sizeof(uint32_t)
                                            : (size_t)rows * (size_t)ntiles * sizeof(unsigned short)));
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

// Largest k and long rows take the finish kernel's shared memory past the default 48 KB: the kernel's
// limit is raised once per device (slot: one per kernel instantiation), not on every call.
constexpr size_t kFinishSmemLimit = 96 * 1024;
static bool raise_smem_limit_once(void (*kern)(const SparsifyParams), int slot, size_t limit) {
    constexpr int kMaxDevices = 64;
    static bool done[12][kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    const bool cached = dev >= 0 && dev < kMaxDevices;
    if (cached && done[slot][dev]) return true;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)limit) != cudaSuccess) return false;
    if (cached) done[slot][dev] = true;
    return true;
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

static int sparsify_impl(const void* logits, int dtype, int B, int gamma, int V, long long row_stride_elems, int k,
                         float top_p, float temperature, int num_samples, const float* uniforms, int* idx, float* logit,
                         int* count, int* token, float* lse, float* mass, double* lse2, void* workspace,
                         size_t workspace_bytes, void* stream) {
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
    p.idx = idx; p.logit = logit; p.count = count; p.token = token; p.lse = lse; p.mass = mass; p.lse2 = lse2;
    p.nshards = 0; p.part_k = 0; p.part_idx = nullptr; p.part_logit = nullptr; p.part_count = nullptr; p.part_lse2 = nullptr;
    p.nchunks = pl.nchunks; p.split = pl.split;
    p.group_log2 = pl.group_log2; p.ngroups = pl.ngroups; p.tile_cap = pl.tile_cap; p.cand_cap = pl.cand_cap;
    p.poll_limit = g_sparsify_poll_limit;
    unsigned char* ws = (unsigned char*)workspace;
    p.status = (int*)ws;
    p.seg_ready = (int*)(ws + pl.ws_ready_off);
    p.seg_stats = (SegStat*)(ws + pl.ws_stats_off);
    p.tile_max = (unsigned short*)(ws + pl.ws_tiles_off);
    p.row_list = (uint32_t*)(ws + pl.ws_tiles_off);
    p.local_bound = pl.local_bound ? 1 : 0;

    cudaStream_t st = (cudaStream_t)stream;
    void (*strm)(const SparsifyParams);
    if (pl.local_bound) strm = dtype == TSLT_F32 ? sparsify_stream_kernel<float, true> : sparsify_stream_kernel<bf16_t, true>;
    else strm = dtype == TSLT_F32 ? sparsify_stream_kernel<float, false> : sparsify_stream_kernel<bf16_t, false>;
    const int strm_slot = (pl.local_bound ? 2 : 0) + (dtype == TSLT_F32 ? 0 : 1);
    if (!prefer_shared_carveout_once(strm, strm_slot)) return TSLT_ERR_CUDA;
    if (pl.stream_smem > 48 * 1024 && !raise_smem_limit_once(strm, 8 + strm_slot, kStreamSmemLimit)) return TSLT_ERR_CUDA;
    strm<<<pl.split.grid, kBlockThreads, pl.stream_smem, st>>>(p);
    if (cudaGetLastError() != cudaSuccess) return TSLT_ERR_CUDA;
    void (*fin)(const SparsifyParams);
    const bool f32 = dtype == TSLT_F32, small = pl.fin_threads == 128;
    if (pl.local_bound) {
        if (small) fin = f32 ? sparsify_finish_kernel<float, 128, true> : sparsify_finish_kernel<bf16_t, 128, true>;
        else fin = f32 ? sparsify_finish_kernel<float, 256, true> : sparsify_finish_kernel<bf16_t, 256, true>;
    } else {
        fin = f32 ? sparsify_finish_kernel<float, kSegmentFinishThreads, false> : sparsify_finish_kernel<bf16_t, kSegmentFinishThreads, false>;
    }
    const int fin_slot = (small ? 0 : 2) + (f32 ? 0 : 1) + (pl.local_bound ? 4 : 0);
    if (!prefer_shared_carveout_once(fin, 4 + fin_slot)) return TSLT_ERR_CUDA;
    if (pl.cand_cap > kListPerThread * pl.fin_threads || k > kWinnersPerThread * pl.fin_threads) return TSLT_ERR_UNSUPPORTED;  // (cannot happen: see finish_threads)
    if (pl.fin_smem > kFinishSmemLimit) return TSLT_ERR_UNSUPPORTED;  // (rows of tens of millions of logits: the line maxima no longer fit)
    if (pl.fin_smem > 48 * 1024 && !raise_smem_limit_once(fin, fin_slot, kFinishSmemLimit)) return TSLT_ERR_CUDA;
    if (launch_dependent(fin, rows, pl.fin_threads, pl.fin_smem, st, p) != cudaSuccess) return TSLT_ERR_CUDA;
    return TSLT_OK;
}

extern "C" int tslt_sparsify(const void* logits, int dtype, int B, int gamma, int V,
                             long long row_stride_elems, int k, float top_p, float temperature,
                             int num_samples, const float* uniforms, int* idx, float* logit, int* count,
                             int* token, float* lse, float* mass, void* workspace, size_t workspace_bytes,
                             void* stream) {
    return sparsify_impl(logits, dtype, B, gamma, V, row_stride_elems, k, top_p, temperature, num_samples, uniforms, idx,
                         logit, count, token, lse, mass, nullptr, workspace, workspace_bytes, stream);
}

extern "C" int tslt_sparsify_shard(const void* logits, int dtype, int rows, int V_shard, long long row_stride_elems, int k,
                                   float temperature, int* idx, float* logit, int* count, double* lse2, void* workspace,
                                   size_t workspace_bytes, void* stream) {
    if (rows > 0 && !lse2) return TSLT_ERR_INVALID_ARG;
    return sparsify_impl(logits, dtype, rows, 1, V_shard, row_stride_elems, k, 1.0f, temperature, 0, nullptr, idx, logit,
                         count, nullptr, nullptr, nullptr, lse2, workspace, workspace_bytes, stream);
}

extern "C" int tslt_sparsify_merge(int dtype, int rows, int nshards, const int* shard_offset, int k, const int* part_idx,
                                   const float* part_logit, const int* part_count, const double* part_lse2, float top_p,
                                   float temperature, int num_samples, const float* uniforms, int* idx, float* logit,
                                   int* count, int* token, float* lse, float* mass, void* workspace,
                                   size_t workspace_bytes, void* stream) {
    if (dtype != TSLT_F32 && dtype != TSLT_BF16) return TSLT_ERR_UNSUPPORTED;
    if (rows < 0 || nshards < 1 || k <= 0 || !shard_offset || !(top_p > 0.0f) || !(temperature > 0.0f) ||
        !isfinite(temperature) || num_samples < 0)
        return TSLT_ERR_INVALID_ARG;
    if (nshards > kMaxShards || k > TSLT_MAX_K || (long long)nshards * k > kMaxMergeList) return TSLT_ERR_UNSUPPORTED;
    if (shard_offset[0] < 0) return TSLT_ERR_INVALID_ARG;
    for (int s = 1; s < nshards; ++s)
        if (shard_offset[s] <= shard_offset[s - 1]) return TSLT_ERR_INVALID_ARG;
    if (rows > 0x7fffffff / 64) return TSLT_ERR_UNSUPPORTED;
    if (rows == 0) return TSLT_OK;
    if (!part_idx || !part_logit || !part_count || !part_lse2 || !idx || !logit || !count || !workspace ||
        (num_samples > 0 && (!uniforms || !token)))
        return TSLT_ERR_INVALID_ARG;
    if (((uintptr_t)workspace & 255)) return TSLT_ERR_INVALID_ARG;
    if (workspace_bytes < (size_t)kWsHeaderBytes) return TSLT_ERR_WORKSPACE;

    SparsifyParams p = {};
    p.rows = rows; p.k = k;
    p.top_p = top_p;
    p.c = make_scale(temperature);
    p.num_samples = num_samples;
    p.uniforms = uniforms;
    p.idx = idx; p.logit = logit; p.count = count; p.token = token; p.lse = lse; p.mass = mass; p.lse2 = nullptr;
    p.cand_cap = nshards * k;
    p.status = (int*)workspace;
    p.nshards = nshards; p.part_k = k;
    p.part_idx = part_idx; p.part_logit = part_logit; p.part_count = part_count; p.part_lse2 = part_lse2;
    for (int s = 0; s < kMaxShards; ++s) p.shard_offset[s] = s < nshards ? shard_offset[s] : 0;
    void (*kern)(const SparsifyParams) = dtype == TSLT_F32 ? sparsify_merge_kernel<float> : sparsify_merge_kernel<bf16_t>;
    const size_t smem = finish_layout(0, 0, p.cand_cap, k, 0, true).total;  // at most 512 + 4096 + 8192 + 16384 bytes
    kern<<<rows, kMergeThreads, smem, (cudaStream_t)stream>>>(p);
    if (cudaGetLastError() != cudaSuccess) return TSLT_ERR_CUDA;
    return TSLT_OK;
}

#ifdef TSLT_STAMPS
// Timeline build only: the stamps of the last tslt_sparsify call, [kStampCtas, kStampSlots] nanoseconds
// (streaming CTA c: slots 0 start, 1 end of its loop, 2 handed over; finish CTA of row r: slots 3 enter,
// 4 row ready, 5 hand-over read, 6 candidates gathered, 7 top-k selected, and slot 0 of entry r + kStampCtas / 2: done).
extern "C" int tslt_debug_stamps_sparsify(void* host, size_t bytes) {
    if (bytes > sizeof(unsigned long long) * kStampCtas * kStampSlots) return TSLT_ERR_INVALID_ARG;
    return cudaMemcpyFromSymbol(host, g_stamps, bytes) == cudaSuccess ? TSLT_OK : TSLT_ERR_CUDA;
}
#endif
