// tslt_verify / tslt_tree_verify / tslt_tree_verify_walk: verifier-side speculative sampling
// against a sparse draft (Algorithm 3; Algorithm 5 along the walk of Algorithm 8).
//
// Every target row that is looked at is read from HBM exactly once, with 16-byte loads that go
// straight to registers (each warp instruction covers 512 contiguous bytes); warps run freely, one
// 2 KB chunk per step.  The streaming pass keeps nothing but one (max, sum) pair per chunk of the
// row, written to the workspace.  A resolve step then turns the chunk partials into each row's
// log-normaliser, rebuilds the sparse q~ in fp64, runs the acceptance tests, and samples the
// correction token from the full-vocabulary residual.  Because q~ is sparse, the residual is
// a multiple of p outside the draft set S and explicit values on S, so its CDF is the chunk
// partials corrected by at most k entries; only the one chunk that holds the sampled token is
// read a second time.
//   tslt_verify, tslt_tree_verify: a streaming kernel over all rows, then (programmatic dependent
//     launch) a resolve kernel with one CTA per sequence.
//   tslt_tree_verify_walk: one launch per tree level; only the row of the node each sequence's
//     walk has reached is streamed, and the CTA that completes it (a ticket counter, no waiting)
//     runs Algorithm 5 at that node and moves the walk on.
#include <math.h>

#include <mutex>
#include <vector>

#include "tslt_common.cuh"
#include "tslt_payload.cuh"
#include "tslt_rowmath.cuh"

namespace tslt {

constexpr int kMaxChunks = 2048;   // chunk partials of one row must fit the resolver's shared memory
// A residual mass at or below this is taken as zero: p is known to the accuracy of the row's fp32
// normaliser (a few 1e-7 relative), so a residual sum max(0, p - q~) this small is rounding noise of
// a draft that equals the target on its support.  Exact arithmetic gives 0 there, and the verifier
// then samples the unmodified p (the fall-back the method's degenerate case takes).
constexpr double kMinResidualMass = 4.0e-7;
constexpr int kMaxTreeNodes = 1024;

struct VerifyParams {
    const unsigned char* logits;
    long long row_stride_bytes;
    int V, B, rows_per_seq, k;
    int nchunks;
    RowSplit split;
    ScaleC cp, cq;
    const int* draft_idx;
    const float* draft_logit;
    const int* draft_count;
    // the drafts as packed uplink records instead (draft_idx == nullptr): [draft rows, pay_words]
    const uint32_t* payload;
    int pay_words, pay_bi, pay_bp, pay_fmt;
    // sequence mode
    int gamma;
    const int* draft_token;
    const float* u_accept;
    const float* u_sample;
    int* accepted_len;
    int* out_token;
    float* accept_prob;
    float* beta_hat;
    float* lse_p;
    // tree mode
    int N, M, max_depth;
    const int* tree_meta;  // child_begin[N+1] | child_list[N-1] | node_draft_row[N]
    const int* node_token;
    int* accepted_path;
    // workspace
    int* status;
    int* tickets;      // path walk only: [levels, B]
    float2* partials;  // [B * rows_per_seq, nchunks]; path walk: [B, nchunks], the row each walk is at
    struct WalkState* walk;  // path walk only: [B]
};

// Where a sequence's walk stands between two levels of tslt_tree_verify_walk.
struct WalkState {
    int node, len, done, pad;
};

struct VerifyShared {
    double scratch[16];
    double slot_a, slot_q;
    int slot_found;
    int ticket;
};

// Resolver work arrays (dynamic shared memory; only the CTA that resolves a sequence uses them).
struct ResolverArrays {
    double* chunkR;  // kMaxChunks
    int* s_idx;      // 1024
    double* s_p;     // 1024
    double* s_a;     // 1024
    double* s_q;     // 1024
    double* r;       // 1024
};
constexpr int kResolverBytes = kMaxChunks * 8 + 1024 * 4 + 4 * 1024 * 8;
constexpr int kVerifyArena = kResolverBytes;
__device__ __forceinline__ ResolverArrays carve(unsigned char* arena) {
    ResolverArrays a;
    a.chunkR = reinterpret_cast<double*>(arena);
    a.s_idx = reinterpret_cast<int*>(arena + kMaxChunks * 8);
    a.s_p = reinterpret_cast<double*>(arena + kMaxChunks * 8 + 4096);
    a.s_a = a.s_p + 1024;
    a.s_q = a.s_a + 1024;
    a.r = a.s_q + 1024;
    return a;
}

__device__ __forceinline__ double accept_probability(double p, double q) {
    if (q > 0.0) {
        const double ratio = p / q;
        return ratio < 1.0 ? ratio : 1.0;
    }
    return p > 0.0 ? 1.0 : 0.0;
}

// base-2 log-normaliser of a row from its chunk partials: L2 = M + log2 sum S_c 2^(M_c - M)
__device__ __forceinline__ double row_log2_norm(const float2* part, int nchunks, int tid, double* scratch) {
    double mx = -INFINITY;
    for (int c = tid; c < nchunks; c += kBlockThreads) {
        const float2 ms = __ldcg(&part[c]);
        if (ms.y > 0.f) mx = fmax(mx, (double)ms.x);
    }
    mx = block_max(mx, tid, scratch);
    double s = 0.0;
    for (int c = tid; c < nchunks; c += kBlockThreads) {
        const float2 ms = __ldcg(&part[c]);
        if (ms.y > 0.f) s += (double)ms.y * exp2((double)ms.x - mx);
    }
    s = block_sum(s, tid, scratch);
    return s > 0.0 ? mx + log2(s) : -INFINITY;
}

// The transmitted pairs of a draft row, from the unpacked arrays or straight from the packed record.
// A record whose count word is not in [0, k] was not written by this library: the row reads as empty
// and TSLT_STATUS_BAD_RECORD is set in the status word.
__device__ __forceinline__ int draft_len(const VerifyParams& p, size_t draft_row) {
    int n;
    if (p.payload) {
        n = (int)__ldg(p.payload + draft_row * (size_t)p.pay_words);
        if (n < 0 || n > p.k) {
            atomicOr(p.status, TSLT_STATUS_BAD_RECORD);
            n = 0;
        }
    } else {
        n = p.draft_count[draft_row];
        n = n < 0 ? 0 : (n > p.k ? p.k : n);
    }
    return n;
}
__device__ __forceinline__ void draft_entry(const VerifyParams& p, size_t draft_row, int i, int* idx, float* logit) {
    if (p.payload) {
        const uint32_t* rec = p.payload + draft_row * (size_t)p.pay_words;
        const int word = 1 + (int)(((long long)i * (p.pay_bi + p.pay_bp)) >> 5);
        const unsigned long long lo = __ldg(rec + word);
        const unsigned long long mid = word + 1 < p.pay_words ? __ldg(rec + word + 1) : 0u;
        const unsigned long long hi = word + 2 < p.pay_words ? __ldg(rec + word + 2) : 0u;
        decode_entry(lo, mid, hi, i, p.pay_bi, p.pay_bp, p.pay_fmt, idx, logit);
    } else {
        *idx = p.draft_idx[draft_row * (size_t)p.k + i];
        *logit = p.draft_logit[draft_row * (size_t)p.k + i];
    }
}

// p(v) of a streamed row.  cs is the scale AS THE STREAMING PASS USED IT (the fp32 rounding of
// log2(e) / T, widened): the row's log-normaliser L2 was accumulated with it, and only the same
// scale in the numerator makes a common offset of the logits cancel exactly.
template <typename T>
__device__ __forceinline__ double token_prob(const unsigned char* rowp, int v, int V, double cs, double L2) {
    if (v < 0 || v >= V || !(L2 > -INFINITY)) return 0.0;
    const float z = Elt<T>::load(rowp, v);
    if (!(fabsf(z) <= 3.4028234e38f)) return 0.0;  // non-finite logit: probability 0
    return exp2((double)z * cs - L2);
}

// Rebuild q~ from the transmitted pairs of one draft row into s_idx / s_q; returns n.
__device__ __forceinline__ int load_draft(const VerifyParams& p, size_t draft_row, const ResolverArrays& A,
                                          int tid, double* scratch) {
    const int n = draft_len(p, draft_row);
    double mx = -INFINITY;
    for (int i = tid; i < n; i += kBlockThreads) {
        int v;
        float l;
        draft_entry(p, draft_row, i, &v, &l);
        A.s_idx[i] = v;
        const bool fin = fabsf(l) <= 3.4028234e38f;
        const double y = fin ? (double)l * p.cq.d : -INFINITY;
        A.s_q[i] = y;
        mx = fmax(mx, y);
    }
    mx = block_max(mx, tid, scratch);
    double w = 0.0;
    for (int i = tid; i < n; i += kBlockThreads) {
        const double y = A.s_q[i];
        const double e = y > -INFINITY ? exp2(y - mx) : 0.0;
        A.s_q[i] = e;
        w += e;
    }
    const double W = block_sum(w, tid, scratch);
    for (int i = tid; i < n; i += kBlockThreads) A.s_q[i] = W > 0.0 ? A.s_q[i] / W : 0.0;
    consumer_sync();
    return n;
}

// Sample one token over the full vocabulary from the weights
//   w(v) = c_out * p(v) for v outside S,   w(idx_i) = s_a[i] for the n entries of S,
// by inverse CDF in ascending index with uniform u.  Returns -1 if the total is not positive.
template <typename T>
__device__ __forceinline__ int sample_full_vocab(const VerifyParams& p, const unsigned char* rowp,
                                                 const float2* part, double L2, double c_out, int n,
                                                 const ResolverArrays& A, float u_raw, int tid,
                                                 VerifyShared* sh) {
    constexpr int kChunkElems = kChunkBytes / Elt<T>::kBytes;
    const int nch = p.nchunks;
    for (int c = tid; c < nch; c += kBlockThreads) {
        const float2 ms = __ldcg(&part[c]);
        A.chunkR[c] = (ms.y > 0.f && L2 > -INFINITY) ? c_out * (double)ms.y * exp2((double)ms.x - L2) : 0.0;
    }
    consumer_sync();
    // entries of S replace c_out * p by their explicit value; one writer per chunk (S is ascending)
    for (int i = tid; i < n; i += kBlockThreads) {
        const int v = A.s_idx[i];
        if (v < 0 || v >= p.V) continue;
        const int c = v / kChunkElems;
        const int vp = i > 0 ? A.s_idx[i - 1] : -1;
        const bool first = !(vp >= 0 && vp < p.V && vp / kChunkElems == c);
        if (first) {
            double acc = 0.0;
            for (int j = i; j < n; ++j) {
                const int vj = A.s_idx[j];
                if (vj < 0 || vj >= p.V || vj / kChunkElems != c) break;
                acc += A.s_a[j] - c_out * A.s_p[j];
            }
            const double val = A.chunkR[c] + acc;
            A.chunkR[c] = val > 0.0 ? val : 0.0;
        }
    }
    consumer_sync();
    block_inclusive_scan(A.chunkR, nch, tid, sh->scratch);
    const double Z = A.chunkR[nch - 1];
    if (!(Z > kMinResidualMass)) {
        consumer_sync();
        return -1;
    }
    const double u = (double)clamp_uniform(u_raw);
    const double target = u * Z;
    int c = first_greater(A.chunkR, nch, target);
    bool take_last = false;
    if (c >= nch) {
        // rounding left nothing above the target: last chunk with positive mass, its last positive item
        c = nch - 1;
        while (c > 0 && !(A.chunkR[c] - A.chunkR[c - 1] > 0.0)) --c;
        take_last = true;
    }
    const double base = c > 0 ? A.chunkR[c - 1] : 0.0;
    const double Rc = A.chunkR[c] - base;
    const double frac = take_last ? 2.0 : (target - base) / Rc;
    consumer_sync();
    // second touch of one chunk: exact weights of its elements
    const int v0 = c * kChunkElems;
    const int ne = min(kChunkElems, p.V - v0);
    for (int e = tid; e < ne; e += kBlockThreads) A.r[e] = c_out * token_prob<T>(rowp, v0 + e, p.V, (double)p.cp.f, L2);
    consumer_sync();
    for (int i = tid; i < n; i += kBlockThreads) {
        const int v = A.s_idx[i];
        if (v >= v0 && v < v0 + ne) A.r[v - v0] = A.s_a[i] > 0.0 ? A.s_a[i] : 0.0;
    }
    consumer_sync();
    // keep the plain weights for the "last positive" fallback, scan a copy in place of chunkR
    double* cumr = A.chunkR;  // chunk table no longer needed
    for (int e = tid; e < ne; e += kBlockThreads) cumr[e] = A.r[e];
    consumer_sync();
    block_inclusive_scan(cumr, ne, tid, sh->scratch);
    const double Rc2 = cumr[ne - 1];
    if (!(Rc2 > 0.0)) {  // the chunk's mass was rounding noise of the corrections: nothing to sample here
        consumer_sync();
        return -1;
    }
    int pos = frac < 1.5 ? first_greater(cumr, ne, frac * Rc2) : ne;
    if (pos >= ne) {
        pos = ne - 1;
        while (pos > 0 && !(A.r[pos] > 0.0)) --pos;
    }
    consumer_sync();
    return v0 + pos;
}

// One warp: base-2 log-normaliser of a row from its chunk partials (warp shuffles only).
__device__ __forceinline__ double row_log2_norm_warp(const float2* part, int nchunks, int lane) {
    // fp64 is scarce (two warp instructions per clock per SM): the per-chunk factors 2^(M_c - M)
    // are taken in fp32 (the exponents are differences of nearby chunk maxima, so the 1-ulp factor
    // errors are ~1e-7 with random sign over hundreds of chunks); the sum is kept in fp64
    constexpr int kHold = 8;  // pairs a lane keeps in registers: rows of up to 256 chunks (512 KB) take one trip to memory
    double mx = -INFINITY, s = 0.0;
    if (nchunks <= 32 * kHold) {
        float2 ms[kHold];
#pragma unroll
        for (int j = 0; j < kHold; ++j) {
            const int c = lane + 32 * j;
            ms[j] = c < nchunks ? __ldcg(&part[c]) : make_float2(0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < kHold; ++j)
            if (ms[j].y > 0.f) mx = fmax(mx, (double)ms[j].x);
        mx = warp_max(mx);
#pragma unroll
        for (int j = 0; j < kHold; ++j)
            if (ms[j].y > 0.f) s += (double)(ms[j].y * exp2f((float)((double)ms[j].x - mx)));
    } else {
#pragma unroll 4
        for (int c = lane; c < nchunks; c += 32) {
            const float2 ms = __ldcg(&part[c]);
            if (ms.y > 0.f) mx = fmax(mx, (double)ms.x);
        }
        mx = warp_max(mx);
#pragma unroll 4
        for (int c = lane; c < nchunks; c += 32) {
            const float2 ms = __ldcg(&part[c]);
            if (ms.y > 0.f) s += (double)(ms.y * exp2f((float)((double)ms.x - mx)));
        }
    }
    s = warp_sum(s);
    double L2 = -INFINITY;
    if (lane == 0 && s > 0.0) L2 = mx + log2(s);  // one lane: a double log2 is ~60 fp64 instructions
    return __shfl_sync(0xffffffffu, L2, 0);
}

// One warp: acceptance probability min(1, p(x) / q~(x)) of one position, and (if wanted) the
// truncated acceptance rate sum_S min(p, q~).  q~ is rebuilt from the transmitted pairs: up to 256
// pairs wait in registers (one trip to memory for them, one for the target logits at their tokens);
// more are read in passes over global memory (at most 8 KB, cache resident).
template <typename T>
__device__ __forceinline__ double position_accept_prob(const VerifyParams& p, size_t draft_row, const unsigned char* rowp,
                                                       double L2, int lane, double* beta_hat_out) {
    const int n = draft_len(p, draft_row);
    const int x = p.draft_token[draft_row];
    constexpr int kHold = 8;  // pairs a lane keeps in registers: up to 256 pairs take one trip to memory
    if (n <= 32 * kHold) {
        const double cs = (double)p.cp.f;
        int v[kHold];
        float l[kHold], zt[kHold];
#pragma unroll
        for (int j = 0; j < kHold; ++j) {
            const int i = lane + 32 * j;
            v[j] = -1;
            l[j] = -INFINITY;
            if (i < n) draft_entry(p, draft_row, i, &v[j], &l[j]);
        }
        const float zx = (x >= 0 && x < p.V) ? Elt<T>::load(rowp, x) : -INFINITY;  // asked for before the pairs are used
        if (beta_hat_out) {
#pragma unroll
            for (int j = 0; j < kHold; ++j) zt[j] = (v[j] >= 0 && v[j] < p.V) ? Elt<T>::load(rowp, v[j]) : -INFINITY;
        }
        double mx = -INFINITY;
#pragma unroll
        for (int j = 0; j < kHold; ++j)
            if (fabsf(l[j]) <= 3.4028234e38f) mx = fmax(mx, (double)l[j] * p.cq.d);
        mx = warp_max(mx);
        double e[kHold], w = 0.0, ex = 0.0;
#pragma unroll
        for (int j = 0; j < kHold; ++j) {
            e[j] = fabsf(l[j]) <= 3.4028234e38f ? exp2((double)l[j] * p.cq.d - mx) : 0.0;
            w += e[j];
            if (lane + 32 * j < n && v[j] == x) ex = e[j];
        }
        const double W = warp_sum(w);
        ex = warp_max(ex);  // the pairs are distinct: at most one lane found x
        const double qx = W > 0.0 ? ex / W : 0.0;
        const bool row_ok = L2 > -INFINITY;
        if (beta_hat_out) {
            double bh = 0.0;
#pragma unroll
            for (int j = 0; j < kHold; ++j) {
                const double pv = (row_ok && fabsf(zt[j]) <= 3.4028234e38f) ? exp2((double)zt[j] * cs - L2) : 0.0;
                if (lane + 32 * j < n) bh += fmin(pv, W > 0.0 ? e[j] / W : 0.0);
            }
            *beta_hat_out = warp_sum(bh);
        }
        const double px = (row_ok && fabsf(zx) <= 3.4028234e38f) ? exp2((double)zx * cs - L2) : 0.0;
        return accept_probability(px, qx);
    }
    // more pairs than a lane holds: passes over the pairs (cache resident after the first)
    double mx = -INFINITY;
    for (int i = lane; i < n; i += 32) {
        int v;
        float l;
        draft_entry(p, draft_row, i, &v, &l);
        if (fabsf(l) <= 3.4028234e38f) mx = fmax(mx, (double)l * p.cq.d);
    }
    mx = warp_max(mx);
    double w = 0.0, ex = 0.0;
    for (int i = lane; i < n; i += 32) {
        int v;
        float l;
        draft_entry(p, draft_row, i, &v, &l);
        const double e = fabsf(l) <= 3.4028234e38f ? exp2((double)l * p.cq.d - mx) : 0.0;
        w += e;
        if (v == x) ex = e;
    }
    const double W = warp_sum(w);
    ex = warp_max(ex);  // the pairs are distinct: at most one lane found x
    const double qx = W > 0.0 ? ex / W : 0.0;
    if (beta_hat_out) {
        double bh = 0.0;
        for (int i = lane; i < n; i += 32) {
            int v;
            float l;
            draft_entry(p, draft_row, i, &v, &l);
            const double e = fabsf(l) <= 3.4028234e38f ? exp2((double)l * p.cq.d - mx) : 0.0;
            bh += fmin(token_prob<T>(rowp, v, p.V, (double)p.cp.f, L2), W > 0.0 ? e / W : 0.0);
        }
        *beta_hat_out = warp_sum(bh);
    }
    return accept_probability(token_prob<T>(rowp, x, p.V, (double)p.cp.f, L2), qx);
}

template <typename T>
__device__ void resolve_sequence(const VerifyParams& p, int b, unsigned char* arena, VerifyShared* sh, int tid) {
    const ResolverArrays A = carve(arena);
    const int gamma = p.gamma;
    const int lane = tid & 31, warp = tid >> 5;
    const size_t r0 = (size_t)b * (gamma + 1);
    // ---- every position on its own warp: log-normaliser of its target row, then its acceptance test
    double* L2s = A.chunkR;               // gamma + 1 entries (gamma < 1024, checked on the host)
    double* aps = A.chunkR + (gamma + 1);  // gamma entries
    // (the bonus row's log-normaliser is only needed if every position is accepted or lse_p is wanted)
    const int j_end = p.lse_p ? gamma + 1 : gamma;
    for (int j = warp; j < j_end; j += kWarps) {
        const float2* part = p.partials + (r0 + j) * (size_t)p.nchunks;
        if (j < gamma) {
            // what the acceptance test will read after the log-normaliser is asked for now: the
            // position's transmitted pairs and the target logit of its drafted token
            const size_t dr = (size_t)b * gamma + j;
            if (p.payload) {
                for (int o = lane * 32; o < p.pay_words; o += 32 * 32)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(p.payload + dr * (size_t)p.pay_words + o));
            } else {
                for (int o = lane * 32; o < p.k; o += 32 * 32) {
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(p.draft_logit + dr * (size_t)p.k + o));
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(p.draft_idx + dr * (size_t)p.k + o));
                }
            }
            if (lane == 0) {
                const int x = p.draft_token[dr];
                if (x >= 0 && x < p.V)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(p.logits + (long long)(r0 + j) * p.row_stride_bytes +
                                                                   (size_t)x * Elt<T>::kBytes));
            }
        }
        const double L2 = row_log2_norm_warp(part, p.nchunks, lane);
        if (lane == 0) {
            L2s[j] = L2;
            if (p.lse_p) p.lse_p[r0 + j] = (float)(L2 * 0.6931471805599453);
        }
        if (j < gamma) {
            const unsigned char* rowp = p.logits + (long long)(r0 + j) * p.row_stride_bytes;
            const size_t dr = (size_t)b * gamma + j;
            double bh = 0.0;
            const double ap = position_accept_prob<T>(p, dr, rowp, L2, lane, p.beta_hat ? &bh : nullptr);
            if (lane == 0) {
                aps[j] = ap;
                if (p.accept_prob) p.accept_prob[dr] = (float)ap;
                if (p.beta_hat) p.beta_hat[dr] = (float)bh;
            }
        }
    }
    consumer_sync();
    TSLT_STAMP(b, 2);
    // ---- the leading run of accepted positions (strict <) ---------------------------------------
    int a = 0;
    while (a < gamma && (double)clamp_uniform(p.u_accept[(size_t)b * gamma + a]) < aps[a]) ++a;
    if (a == gamma && !p.lse_p) {  // all accepted: now the bonus row is needed (uniform branch)
        const double L2 = row_log2_norm_warp(p.partials + (r0 + gamma) * (size_t)p.nchunks, p.nchunks, lane);
        if (tid == 0) L2s[gamma] = L2;
        consumer_sync();
    }
    const double L2_stop = L2s[a];
    consumer_sync();  // chunkR is reused below
    // correction token: residual of the rejected position, or the bonus row
    const unsigned char* rowp = p.logits + (long long)(r0 + a) * p.row_stride_bytes;
    const float2* part = p.partials + (r0 + a) * (size_t)p.nchunks;
    int n = 0;
    if (a < gamma) {
        n = load_draft(p, (size_t)b * gamma + a, A, tid, sh->scratch);
        for (int i = tid; i < n; i += kBlockThreads) {
            const double pv = token_prob<T>(rowp, A.s_idx[i], p.V, (double)p.cp.f, L2_stop);
            A.s_p[i] = pv;
            const double d = pv - A.s_q[i];
            A.s_a[i] = d > 0.0 ? d : 0.0;
        }
        consumer_sync();
    }
    TSLT_STAMP(b, 3);
    const float u = p.u_sample[b];
    int tok = sample_full_vocab<T>(p, rowp, part, L2_stop, 1.0, n, A, u, tid, sh);
    TSLT_STAMP(b, 4);
    if (tok < 0 && n > 0) tok = sample_full_vocab<T>(p, rowp, part, L2_stop, 1.0, 0, A, u, tid, sh);  // degenerate residual
    if (tid == 0) {
        p.accepted_len[b] = a;
        p.out_token[b] = tok;
    }
}

// Algorithm 5 at one node of sequence b's walk (Algorithm 8): `part` holds the chunk partials of the
// node's target row.  Returns the accepted child, where the walk goes on, or -1 if the walk stops
// at this node, *tok_out then being the final token (a leaf's bonus token, or a sample of p^(k+1)).
template <typename T>
__device__ int resolve_tree_node(const VerifyParams& p, int b, int node, const float2* part, const ResolverArrays& A,
                                 VerifyShared* sh, int tid, int* tok_out) {
    const int N = p.N;
    const int* child_begin = p.tree_meta;
    const int* child_list = p.tree_meta + (N + 1);
    const int* node_draft_row = p.tree_meta + (N + 1) + (N - 1);
    const size_t r = (size_t)b * N + node;
    const unsigned char* rowp = p.logits + (long long)r * p.row_stride_bytes;
    const double L2 = row_log2_norm(part, p.nchunks, tid, sh->scratch);
    const int dr = node_draft_row[node];
    const float u = p.u_sample[r];
    if (dr < 0) {
        *tok_out = sample_full_vocab<T>(p, rowp, part, L2, 1.0, 0, A, u, tid, sh);  // leaf: bonus from its own row
        return -1;
    }
    const int n = load_draft(p, (size_t)b * p.M + dr, A, tid, sh->scratch);
    double ps = 0.0;
    for (int i = tid; i < n; i += kBlockThreads) {
        const double pv = token_prob<T>(rowp, A.s_idx[i], p.V, (double)p.cp.f, L2);
        A.s_p[i] = pv;
        A.s_a[i] = pv;
        ps += pv;
    }
    const double PS = block_sum(ps, tid, sh->scratch);
    const double out_mass = 1.0 - PS > 0.0 ? 1.0 - PS : 0.0;  // mass of p outside S
    double c_out = 1.0;
    for (int ci = child_begin[node]; ci < child_begin[node + 1]; ++ci) {
        const int c = child_list[ci];
        const int x = p.node_token[(size_t)b * N + c];
        if (tid == 0) sh->slot_found = 0;
        consumer_sync();
        for (int i = tid; i < n; i += kBlockThreads)
            if (A.s_idx[i] == x) {
                sh->slot_a = A.s_a[i];
                sh->slot_q = A.s_q[i];
                sh->slot_found = 1;
            }
        consumer_sync();
        double pa, qx;
        if (sh->slot_found) {
            pa = sh->slot_a;
            qx = sh->slot_q;
        } else {
            pa = c_out * token_prob<T>(rowp, x, p.V, (double)p.cp.f, L2);
            qx = 0.0;
        }
        const double ap = accept_probability(pa, qx);
        const double rr = (double)clamp_uniform(p.u_accept[(size_t)b * N + c]);
        if (rr < ap) {
            consumer_sync();
            return c;
        }
        // rejected: p^(i+1) = norm(max(0, p^(i) - q~)), on S explicitly, elsewhere by the scalar
        double zs = 0.0;
        for (int i = tid; i < n; i += kBlockThreads) {
            const double d = A.s_a[i] - A.s_q[i];
            zs += d > 0.0 ? d : 0.0;
        }
        const double Z = block_sum(zs, tid, sh->scratch) + c_out * out_mass;
        if (Z > kMinResidualMass) {
            for (int i = tid; i < n; i += kBlockThreads) {
                const double d = A.s_a[i] - A.s_q[i];
                A.s_a[i] = d > 0.0 ? d / Z : 0.0;
            }
            c_out /= Z;
        }
        consumer_sync();
    }
    int tok = sample_full_vocab<T>(p, rowp, part, L2, c_out, n, A, u, tid, sh);
    if (tok < 0) tok = sample_full_vocab<T>(p, rowp, part, L2, 1.0, 0, A, u, tid, sh);
    *tok_out = tok;
    return -1;
}

// The whole walk of one sequence when every node's row has been streamed (tslt_tree_verify).
template <typename T>
__device__ void resolve_tree(const VerifyParams& p, int b, unsigned char* arena, VerifyShared* sh, int tid) {
    const ResolverArrays A = carve(arena);
    int* path = p.accepted_path + (size_t)b * p.max_depth;
    for (int d = tid; d < p.max_depth; d += kBlockThreads) path[d] = -1;
    consumer_sync();
    int node = 0, len = 0, tok = -1;
    for (int depth = 0; depth <= p.max_depth; ++depth) {
        const float2* part = p.partials + ((size_t)b * p.N + node) * (size_t)p.nchunks;
        const int next = resolve_tree_node<T>(p, b, node, part, A, sh, tid, &tok);
        if (next < 0) break;
        if (len < p.max_depth && tid == 0) path[len] = next;
        ++len;
        node = next;
    }
    if (tid == 0) {
        p.accepted_len[b] = len;
        p.out_token[b] = tok;
    }
}

// Streaming pass over chunks [chunk_begin, chunk_end) of the row at rowp: (max, sum) of every chunk,
// the chunk's own maximum as the reference exponent, into part[chunk].
template <typename T>
__device__ __forceinline__ void stream_chunks(const VerifyParams& p, const unsigned char* rowp, float2* part,
                                              int chunk_begin, int chunk_end, int lane, int warp) {
    const RowExtent ext = row_extent<T>(p.V);
    const float c = p.cp.f;
    for (int ch = chunk_begin + warp; ch < chunk_end; ch += kWarps) {
        LaneTile<T> lt;
        lt.load(rowp, ch * kVecsPerChunk, lane, ext);
        const float wm = warp_max(lt.reduce_max());
        LaneSum ls;
        ls.reset();
        if (wm > -INFINITY) ls.M = wm * c;
        lt.accumulate(ls, c);
        const float Sw = warp_sum(ls.total());
        if (lane == 0) part[ch] = make_float2(ls.M, Sw);
    }
}

constexpr int kStreamCtasPerSm = 6;  // streaming-only kernel: 40 registers per thread, no shared memory

// First launch: the streaming pass alone (no shared memory, no ticket, no fence: the kernel boundary
// publishes the partials).  Block 0 clears the workspace's status word before it lets the resolve
// kernel be scheduled, so the word never carries over from an earlier call.
template <typename T>
__global__ void __launch_bounds__(kBlockThreads, kStreamCtasPerSm) verify_stream_kernel(const VerifyParams p) {
    if (blockIdx.x == 0) {
        if (threadIdx.x == 0) {
            *(volatile int*)p.status = 0;
            __threadfence();
        }
        __syncthreads();
    }
    allow_dependent_launch();
    const RowWork wk = locate_work(p.split, blockIdx.x, p.nchunks);
    stream_chunks<T>(p, p.logits + (long long)wk.row * p.row_stride_bytes, p.partials + (size_t)wk.row * p.nchunks,
                     wk.chunk_begin, wk.chunk_end, threadIdx.x & 31, threadIdx.x >> 5);
}
// Second launch: one CTA per sequence resolves it.
template <typename T, bool kTree>
__global__ void __launch_bounds__(kBlockThreads, 4) verify_resolve_kernel(const VerifyParams p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned char* arena = smem_raw;  // plain offsets only: keeps the shared address space
    VerifyShared* sh = reinterpret_cast<VerifyShared*>(arena + kVerifyArena);
    TSLT_STAMP(blockIdx.x, 0);
    wait_for_primary_kernel();  // the partials come from the streaming kernel
    TSLT_STAMP(blockIdx.x, 1);
    if (kTree) resolve_tree<T>(p, blockIdx.x, arena, sh, threadIdx.x);
    else resolve_sequence<T>(p, blockIdx.x, arena, sh, threadIdx.x);
}

// One level of the path walk: every sequence whose walk is still going has the row of its current
// node streamed by the CTAs of its segments; the CTA that completes the row (a ticket counter: the
// last to arrive carries on, nobody waits) runs Algorithm 5 at the node and either moves the walk
// to the accepted child or ends it with the final token.  Launched once per tree level, in stream
// order; the walk state, zeroed on the stream before the first level, carries over in the workspace.
template <typename T>
__global__ void __launch_bounds__(kBlockThreads, 4) tree_walk_level_kernel(const VerifyParams p, int level) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned char* arena = smem_raw;
    VerifyShared* sh = reinterpret_cast<VerifyShared*>(arena + kVerifyArena);
    const int tid = threadIdx.x;
    const RowWork wk = locate_work(p.split, blockIdx.x, p.nchunks);  // "row" = sequence
    const int b = wk.row;
    WalkState* ws = p.walk + b;
    if (__ldcg(&ws->done)) return;  // (the same for every thread of the CTA)
    const int node = __ldcg(&ws->node), len = __ldcg(&ws->len);
    float2* part = p.partials + (size_t)b * p.nchunks;
    stream_chunks<T>(p, p.logits + (long long)((size_t)b * p.N + node) * p.row_stride_bytes, part, wk.chunk_begin,
                     wk.chunk_end, tid & 31, tid >> 5);
    // (the barrier orders every warp's partials before thread 0's fence, which publishes them)
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        sh->ticket = atomicAdd(&p.tickets[(size_t)level * p.B + b], 1);
    }
    __syncthreads();
    if (sh->ticket != wk.nseg - 1) return;
    __threadfence();
    const ResolverArrays A = carve(arena);
    int* path = p.accepted_path + (size_t)b * p.max_depth;
    if (level == 0)
        for (int d = tid; d < p.max_depth; d += kBlockThreads) path[d] = -1;
    int tok = -1;
    const int next = resolve_tree_node<T>(p, b, node, part, A, sh, tid, &tok);
    if (tid == 0) {
        if (next >= 0) {
            if (len < p.max_depth) path[len] = next;
            ws->node = next;
            ws->len = len + 1;
        } else {
            ws->done = 1;
            p.accepted_len[b] = len;
            p.out_token[b] = tok;
        }
    }
}

// ---- host side -------------------------------------------------------------------------------

struct VerifyPlan {
    int nchunks;
    RowSplit split;
    size_t smem;
    size_t ws_state_off, ws_tickets_off, ws_meta_off, ws_partials_off, ws_bytes;
    size_t ws_clear_bytes;  // path walk: what is zeroed on the stream before the first level (state, tickets)
};

static int sm_count_v() {
    static int sms = 0;
    if (sms == 0) {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 148;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
        sms = v;
    }
    return sms;
}

// rows_streamed: rows the streaming pass covers per launch (all target rows; B for the path walk).
// levels > 0: the path walk, with its state and one ticket counter per sequence and level.
static VerifyPlan make_verify_plan(int B, long long rows_streamed, int V, int elt_bytes, int meta_ints, int levels) {
    VerifyPlan pl;
    const long long row_bytes = (long long)V * elt_bytes;
    pl.nchunks = (int)((row_bytes + kChunkBytes - 1) / kChunkBytes);
    // Rows that fill the machine are cut into 64 KB segments; fewer rows into as many segments as give
    // every CTA slot about two CTAs, a segment keeping at least one chunk per warp.
    const int slots = (levels > 0 ? 4 : kStreamCtasPerSm) * sm_count_v();
    int nseg;
    if (rows_streamed >= slots) {
        nseg = (pl.nchunks + 31) / 32;
    } else {
        nseg = (int)((2LL * slots + rows_streamed - 1) / (rows_streamed > 0 ? rows_streamed : 1));
        const int by_len = pl.nchunks / kWarps;
        if (nseg > by_len) nseg = by_len;
        if (nseg > 64) nseg = 64;
    }
    if (nseg < 1) nseg = 1;
    int cps = (pl.nchunks + nseg - 1) / nseg;
    if (cps < 1) cps = 1;
    pl.split.rows = (int)rows_streamed;
    pl.split.cps = cps;
    pl.split.nseg = (pl.nchunks + cps - 1) / cps;
    pl.split.grid = pl.split.rows * pl.split.nseg;
    pl.smem = kVerifyArena + sizeof(VerifyShared) + 256;
    size_t off = kWsHeaderBytes;
    pl.ws_state_off = off;
    if (levels > 0) off = align_up256(off + (size_t)B * sizeof(WalkState));
    pl.ws_tickets_off = off;
    if (levels > 0) off = align_up256(off + (size_t)levels * B * sizeof(int));
    pl.ws_clear_bytes = off;
    pl.ws_meta_off = off;
    off = align_up256(off + (size_t)meta_ints * sizeof(int));
    pl.ws_partials_off = off;
    off = align_up256(off + (size_t)rows_streamed * pl.nchunks * sizeof(float2));
    pl.ws_bytes = off;
    return pl;
}

ScaleC make_scale(float temperature);  // defined with the sparsify launcher

static int check_common(const void* logits, int dtype, int V, long long row_stride_elems, int k,
                        float tq, float tp, const void* workspace) {
    if (dtype != TSLT_F32 && dtype != TSLT_BF16) return TSLT_ERR_UNSUPPORTED;
    const int eb = dtype == TSLT_F32 ? 4 : 2;
    if (V <= 0 || k <= 0 || k > V || !(tq > 0.f) || !(tp > 0.f) || !isfinite(tq) || !isfinite(tp))
        return TSLT_ERR_INVALID_ARG;
    if (k > TSLT_MAX_K) return TSLT_ERR_UNSUPPORTED;
    if ((long long)V * eb > (long long)kMaxChunks * kChunkBytes) return TSLT_ERR_UNSUPPORTED;
    if (!logits || !workspace) return TSLT_ERR_INVALID_ARG;
    if (row_stride_elems < V || ((uintptr_t)logits & 15) || ((row_stride_elems * eb) & 15) ||
        ((uintptr_t)workspace & 255))
        return TSLT_ERR_INVALID_ARG;
    return TSLT_OK;
}

// The resolver's shared memory exceeds the default limit: raise the kernel's limit once per device
// (slot: one per kernel instantiation), not on every call.
template <typename K> static bool raise_smem_limit_once(K kern, int slot, size_t bytes) {
    constexpr int kMaxDevices = 64;
    static bool done[8][kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    const bool cached = dev >= 0 && dev < kMaxDevices;
    if (cached && done[slot][dev]) return true;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) return false;
    if (cached) done[slot][dev] = true;
    return true;
}

template <bool kTree>
static int launch_verify(VerifyParams& p, const VerifyPlan& pl, int dtype, cudaStream_t st) {
    auto resolve = dtype == TSLT_F32 ? verify_resolve_kernel<float, kTree> : verify_resolve_kernel<bf16_t, kTree>;
    if (!raise_smem_limit_once(resolve, (kTree ? 2 : 0) + (dtype == TSLT_F32 ? 0 : 1), pl.smem)) return TSLT_ERR_CUDA;
    if (!prefer_shared_carveout_once(resolve, 8 + (kTree ? 2 : 0) + (dtype == TSLT_F32 ? 0 : 1))) return TSLT_ERR_CUDA;
    if (!(dtype == TSLT_F32 ? prefer_shared_carveout_once(verify_stream_kernel<float>, 12)
                            : prefer_shared_carveout_once(verify_stream_kernel<bf16_t>, 13)))
        return TSLT_ERR_CUDA;
    if (dtype == TSLT_F32) verify_stream_kernel<float><<<(unsigned)pl.split.grid, kBlockThreads, 0, st>>>(p);
    else verify_stream_kernel<bf16_t><<<(unsigned)pl.split.grid, kBlockThreads, 0, st>>>(p);
    if (cudaGetLastError() != cudaSuccess) return TSLT_ERR_CUDA;
    return launch_dependent(resolve, (unsigned)p.B, kBlockThreads, pl.smem, st, p) == cudaSuccess ? TSLT_OK : TSLT_ERR_CUDA;
}

// Host check of the tree arrays and the child lists in the form the kernels read:
// child_begin[N+1] | child_list[N-1] | node_draft_row[N].  Returns the tree's depth, or -1.
static int build_tree_meta(int N, int M, const int* parent, const int* node_draft_row, std::vector<int>& meta) {
    if (parent[0] != -1) return -1;
    std::vector<int> nchild(N, 0), depth(N, 0);
    int maxd = 0;
    for (int n = 1; n < N; ++n) {
        if (parent[n] < 0 || parent[n] >= n) return -1;
        nchild[parent[n]]++;
        depth[n] = depth[parent[n]] + 1;
        if (depth[n] > maxd) maxd = depth[n];
    }
    for (int n = 0; n < N; ++n) {
        const bool internal = nchild[n] > 0;
        if (internal != (node_draft_row[n] >= 0)) return -1;
        if (node_draft_row[n] >= M) return -1;
    }
    meta.assign(3 * (size_t)N, 0);
    int* child_begin = meta.data();
    int* child_list = meta.data() + (N + 1);
    int* ndr = meta.data() + (N + 1) + (N - 1);
    child_begin[0] = 0;
    for (int n = 0; n < N; ++n) child_begin[n + 1] = child_begin[n] + nchild[n];
    std::vector<int> fill(child_begin, child_begin + N);
    for (int n = 1; n < N; ++n) child_list[fill[parent[n]]++] = n;
    for (int n = 0; n < N; ++n) ndr[n] = node_draft_row[n];
    return maxd;
}

}  // namespace tslt

using namespace tslt;

extern "C" int tslt_verify_workspace_bytes(int B, int gamma, int V, int k, size_t* bytes) {
    if (!bytes || B < 0 || gamma < 0 || V <= 0 || k <= 0 || k > V || k > TSLT_MAX_K) return TSLT_ERR_INVALID_ARG;
    VerifyPlan a = make_verify_plan(B, (long long)B * (gamma + 1), V, 2, 0, 0),
               b = make_verify_plan(B, (long long)B * (gamma + 1), V, 4, 0, 0);
    *bytes = a.ws_bytes > b.ws_bytes ? a.ws_bytes : b.ws_bytes;
    return TSLT_OK;
}

// The drafts come either as the arrays tslt_sparsify writes (payload == nullptr) or as packed records.
static int verify_impl(const void* target_logits, int dtype, int B, int gamma, int V, long long row_stride_elems, int k,
                       const int* draft_idx, const float* draft_logit, const int* draft_count,
                       const unsigned int* payload, int prob_format, const int* draft_token, float draft_temperature,
                       float target_temperature, const float* u_accept, const float* u_sample, int* accepted_len,
                       int* out_token, float* accept_prob, float* beta_hat, float* lse_p, void* workspace,
                       size_t workspace_bytes, void* stream) {
    if (B < 0 || gamma < 0) return TSLT_ERR_INVALID_ARG;
    int bi = 0, bp = 0, words = 0;
    if (payload && (V <= 0 || k <= 0 || k > TSLT_MAX_K || !payload_shape(k, V, prob_format, &bi, &bp, &words)))
        return V <= 0 || k <= 0 ? TSLT_ERR_INVALID_ARG : TSLT_ERR_UNSUPPORTED;
    if (B == 0) return TSLT_OK;
    int rc = check_common(target_logits, dtype, V, row_stride_elems, k, draft_temperature, target_temperature,
                          workspace);
    if (rc != TSLT_OK) return rc;
    if (!u_sample || !accepted_len || !out_token ||
        (gamma > 0 && ((!payload && (!draft_idx || !draft_logit || !draft_count)) || !draft_token || !u_accept)))
        return TSLT_ERR_INVALID_ARG;
    if ((long long)B * (gamma + 1) > 0x7fffffffLL / 16 || gamma >= 1024) return TSLT_ERR_UNSUPPORTED;
    const int eb = dtype == TSLT_F32 ? 4 : 2;
    VerifyPlan pl = make_verify_plan(B, (long long)B * (gamma + 1), V, eb, 0, 0);
    if (workspace_bytes < pl.ws_bytes) return TSLT_ERR_WORKSPACE;
    VerifyParams p = {};
    p.logits = (const unsigned char*)target_logits;
    p.row_stride_bytes = row_stride_elems * eb;
    p.V = V; p.B = B; p.rows_per_seq = gamma + 1; p.k = k;
    p.nchunks = pl.nchunks; p.split = pl.split;
    p.cp = make_scale(target_temperature);
    p.cq = make_scale(draft_temperature);
    p.draft_idx = draft_idx; p.draft_logit = draft_logit; p.draft_count = draft_count;
    p.payload = payload; p.pay_words = words; p.pay_bi = bi; p.pay_bp = bp; p.pay_fmt = prob_format;
    p.gamma = gamma; p.draft_token = draft_token; p.u_accept = u_accept; p.u_sample = u_sample;
    p.accepted_len = accepted_len; p.out_token = out_token;
    p.accept_prob = accept_prob; p.beta_hat = beta_hat; p.lse_p = lse_p;
    unsigned char* ws = (unsigned char*)workspace;
    p.status = (int*)ws;
    p.partials = (float2*)(ws + pl.ws_partials_off);
    return launch_verify<false>(p, pl, dtype, (cudaStream_t)stream);
}

extern "C" int tslt_verify(const void* target_logits, int dtype, int B, int gamma, int V,
                           long long row_stride_elems, int k, const int* draft_idx, const float* draft_logit,
                           const int* draft_count, const int* draft_token, float draft_temperature,
                           float target_temperature, const float* u_accept, const float* u_sample,
                           int* accepted_len, int* out_token, float* accept_prob, float* beta_hat,
                           float* lse_p, void* workspace, size_t workspace_bytes, void* stream) {
    return verify_impl(target_logits, dtype, B, gamma, V, row_stride_elems, k, draft_idx, draft_logit, draft_count, nullptr,
                       0, draft_token, draft_temperature, target_temperature, u_accept, u_sample, accepted_len, out_token,
                       accept_prob, beta_hat, lse_p, workspace, workspace_bytes, stream);
}

extern "C" int tslt_verify_packed(const void* target_logits, int dtype, int B, int gamma, int V,
                                  long long row_stride_elems, int k, const unsigned int* payload, int prob_format,
                                  const int* draft_token, float draft_temperature, float target_temperature,
                                  const float* u_accept, const float* u_sample, int* accepted_len, int* out_token,
                                  float* accept_prob, float* beta_hat, float* lse_p, void* workspace,
                                  size_t workspace_bytes, void* stream) {
    if (B > 0 && gamma > 0 && !payload) return TSLT_ERR_INVALID_ARG;
    static const unsigned int kNoRecords = 0;  // gamma == 0: nothing is read, but the packed path is still taken
    return verify_impl(target_logits, dtype, B, gamma, V, row_stride_elems, k, nullptr, nullptr, nullptr,
                       payload ? payload : &kNoRecords, prob_format, draft_token, draft_temperature, target_temperature,
                       u_accept, u_sample, accepted_len, out_token, accept_prob, beta_hat, lse_p, workspace,
                       workspace_bytes, stream);
}

// ---- tslt_verify_static: the same verification with the scratch memory built into the library ----
// Scratch of the no-allocation entry point: ticket counters and per-chunk partial sums.  Every
// GPU that loads the library carries this array until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[TSLT_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device.  In host code the array's name is only
// a handle for the runtime, not an address a kernel could use, so the address is asked for once
// per device (with that device current) and remembered.
static int static_scratch_address(void** out) {
    constexpr int kMaxDevices = 64;
    static void* cache[kMaxDevices] = {};
    static std::mutex mu;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TSLT_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!cache[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return TSLT_ERR_CUDA;
        cache[dev] = ptr;
    }
    *out = cache[dev];
    return TSLT_OK;
}

extern "C" int tslt_verify_static(const void* target_logits, int dtype, int B, int gamma, int V,
                                  long long row_stride_elems, int k, const int* draft_idx,
                                  const float* draft_logit, const int* draft_count, const int* draft_token,
                                  float draft_temperature, float target_temperature, const float* u_accept,
                                  const float* u_sample, int* accepted_len, int* out_token, float* accept_prob,
                                  float* beta_hat, float* lse_p, void* stream) {
    // the size the ordinary entry point would ask a workspace for; too much is refused before
    // anything touches the device
    if (dtype != TSLT_F32 && dtype != TSLT_BF16) return TSLT_ERR_UNSUPPORTED;
    if (B < 0 || gamma < 0 || V <= 0 || k <= 0 || k > V) return TSLT_ERR_INVALID_ARG;
    if (k > TSLT_MAX_K || (long long)B * (gamma + 1) > 0x7fffffffLL / 16) return TSLT_ERR_UNSUPPORTED;
    const size_t need = make_verify_plan(B, (long long)B * (gamma + 1), V, dtype == TSLT_F32 ? 4 : 2, 0, 0).ws_bytes;
    if (need > (size_t)TSLT_STATIC_SCRATCH_BYTES) return TSLT_ERR_STATIC_SCRATCH;
    if (B == 0) return TSLT_OK;
    void* scratch = nullptr;
    const int rs = static_scratch_address(&scratch);
    if (rs != TSLT_OK) return rs;
    // tslt_verify's first kernel clears the status word, and nothing else in the array is read before
    // it has been written, so whatever the previous call left there does no harm
    return tslt_verify(target_logits, dtype, B, gamma, V, row_stride_elems, k, draft_idx, draft_logit, draft_count,
                       draft_token, draft_temperature, target_temperature, u_accept, u_sample, accepted_len,
                       out_token, accept_prob, beta_hat, lse_p, scratch, (size_t)TSLT_STATIC_SCRATCH_BYTES, stream);
}

// levels the path walk can need for a tree of N nodes: one per node on a root-to-leaf path
static int walk_levels_bound(int N) { return N; }

extern "C" int tslt_tree_verify_workspace_bytes(int B, int N, int V, int k, size_t* bytes) {
    if (!bytes || B < 0 || N <= 0 || N > kMaxTreeNodes || V <= 0 || k <= 0 || k > V || k > TSLT_MAX_K)
        return TSLT_ERR_INVALID_ARG;
    VerifyPlan a = make_verify_plan(B, (long long)B * N, V, 2, 3 * N, 0), b = make_verify_plan(B, (long long)B * N, V, 4, 3 * N, 0);
    *bytes = a.ws_bytes > b.ws_bytes ? a.ws_bytes : b.ws_bytes;
    return TSLT_OK;
}

extern "C" int tslt_tree_verify_walk_workspace_bytes(int B, int N, int V, int k, size_t* bytes) {
    if (!bytes || B < 0 || N <= 0 || N > kMaxTreeNodes || V <= 0 || k <= 0 || k > V || k > TSLT_MAX_K)
        return TSLT_ERR_INVALID_ARG;
    VerifyPlan a = make_verify_plan(B, B, V, 2, 3 * N, walk_levels_bound(N)), b = make_verify_plan(B, B, V, 4, 3 * N, walk_levels_bound(N));
    *bytes = a.ws_bytes > b.ws_bytes ? a.ws_bytes : b.ws_bytes;
    return TSLT_OK;
}

// Both tree entry points: walk = false streams every node's row and walks afterwards; walk = true
// streams, level by level, only the rows the walks reach.
static int tree_verify_impl(bool walk, const void* target_logits, int dtype, int B, int N, int V,
                            long long row_stride_elems, const int* parent, const int* node_draft_row, int M, int k,
                            const int* node_token, const int* draft_idx, const float* draft_logit,
                            const int* draft_count, const unsigned int* payload, int prob_format,
                            float draft_temperature, float target_temperature,
                            const float* u_accept, const float* u_sample, int max_depth, int* accepted_path,
                            int* accepted_len, int* out_token, void* workspace, size_t workspace_bytes, void* stream) {
    if (B < 0 || N <= 0 || M < 0 || max_depth < 0 || !parent || !node_draft_row) return TSLT_ERR_INVALID_ARG;
    int bi = 0, bp = 0, words = 0;
    if (payload && (V <= 0 || k <= 0 || k > TSLT_MAX_K || !payload_shape(k, V, prob_format, &bi, &bp, &words)))
        return V <= 0 || k <= 0 ? TSLT_ERR_INVALID_ARG : TSLT_ERR_UNSUPPORTED;
    if (N > kMaxTreeNodes) return TSLT_ERR_UNSUPPORTED;
    std::vector<int> meta;
    const int depth = build_tree_meta(N, M, parent, node_draft_row, meta);  // tree structure, checked on the host
    if (depth < 0 || depth > max_depth) return TSLT_ERR_INVALID_ARG;
    if (B == 0) return TSLT_OK;
    int rc = check_common(target_logits, dtype, V, row_stride_elems, k, draft_temperature, target_temperature,
                          workspace);
    if (rc != TSLT_OK) return rc;
    if (!u_sample || !accepted_len || !out_token || (max_depth > 0 && !accepted_path) ||
        (N > 1 && (!node_token || !u_accept)) || (M > 0 && !payload && (!draft_idx || !draft_logit || !draft_count)))
        return TSLT_ERR_INVALID_ARG;
    if ((long long)B * N > 0x7fffffffLL / 64) return TSLT_ERR_UNSUPPORTED;
    const int eb = dtype == TSLT_F32 ? 4 : 2;
    const int levels = depth + 1;  // nodes on the longest root-to-leaf path
    VerifyPlan pl = walk ? make_verify_plan(B, B, V, eb, 3 * N, walk_levels_bound(N))
                         : make_verify_plan(B, (long long)B * N, V, eb, 3 * N, 0);
    if (workspace_bytes < pl.ws_bytes) return TSLT_ERR_WORKSPACE;

    VerifyParams p = {};
    p.logits = (const unsigned char*)target_logits;
    p.row_stride_bytes = row_stride_elems * eb;
    p.V = V; p.B = B; p.rows_per_seq = N; p.k = k;
    p.nchunks = pl.nchunks; p.split = pl.split;
    p.cp = make_scale(target_temperature);
    p.cq = make_scale(draft_temperature);
    p.draft_idx = draft_idx; p.draft_logit = draft_logit; p.draft_count = draft_count;
    p.payload = payload; p.pay_words = words; p.pay_bi = bi; p.pay_bp = bp; p.pay_fmt = prob_format;
    p.u_accept = u_accept; p.u_sample = u_sample;
    p.accepted_len = accepted_len; p.out_token = out_token;
    p.N = N; p.M = M; p.max_depth = max_depth;
    p.node_token = node_token; p.accepted_path = accepted_path;
    unsigned char* ws = (unsigned char*)workspace;
    p.status = (int*)ws;
    p.walk = (WalkState*)(ws + pl.ws_state_off);
    p.tickets = (int*)(ws + pl.ws_tickets_off);
    p.tree_meta = (const int*)(ws + pl.ws_meta_off);
    p.partials = (float2*)(ws + pl.ws_partials_off);
    cudaStream_t st = (cudaStream_t)stream;
    // pageable source: the runtime stages it before returning, so `meta` may go out of scope
    if (cudaMemcpyAsync(ws + pl.ws_meta_off, meta.data(), meta.size() * sizeof(int), cudaMemcpyHostToDevice, st) !=
        cudaSuccess)
        return TSLT_ERR_CUDA;
    if (!walk) return launch_verify<true>(p, pl, dtype, st);
    // status word, walk state (node 0, length 0, not done) and ticket counters start at zero
    if (cudaMemsetAsync(ws, 0, pl.ws_clear_bytes, st) != cudaSuccess) return TSLT_ERR_CUDA;
    auto kern = dtype == TSLT_F32 ? tree_walk_level_kernel<float> : tree_walk_level_kernel<bf16_t>;
    if (!raise_smem_limit_once(kern, 4 + (dtype == TSLT_F32 ? 0 : 1), pl.smem)) return TSLT_ERR_CUDA;
    for (int level = 0; level < levels; ++level) {
        kern<<<(unsigned)pl.split.grid, kBlockThreads, pl.smem, st>>>(p, level);
        if (cudaGetLastError() != cudaSuccess) return TSLT_ERR_CUDA;
    }
    return TSLT_OK;
}

extern "C" int tslt_tree_verify(const void* target_logits, int dtype, int B, int N, int V,
                                long long row_stride_elems, const int* parent, const int* node_draft_row,
                                int M, int k, const int* node_token, const int* draft_idx,
                                const float* draft_logit, const int* draft_count, float draft_temperature,
                                float target_temperature, const float* u_accept, const float* u_sample,
                                int max_depth, int* accepted_path, int* accepted_len, int* out_token,
                                void* workspace, size_t workspace_bytes, void* stream) {
    return tree_verify_impl(false, target_logits, dtype, B, N, V, row_stride_elems, parent, node_draft_row, M, k,
                            node_token, draft_idx, draft_logit, draft_count, nullptr, 0, draft_temperature, target_temperature,
                            u_accept, u_sample, max_depth, accepted_path, accepted_len, out_token, workspace,
                            workspace_bytes, stream);
}

extern "C" int tslt_tree_verify_walk(const void* target_logits, int dtype, int B, int N, int V,
                                     long long row_stride_elems, const int* parent, const int* node_draft_row,
                                     int M, int k, const int* node_token, const int* draft_idx,
                                     const float* draft_logit, const int* draft_count, float draft_temperature,
                                     float target_temperature, const float* u_accept, const float* u_sample,
                                     int max_depth, int* accepted_path, int* accepted_len, int* out_token,
                                     void* workspace, size_t workspace_bytes, void* stream) {
    return tree_verify_impl(true, target_logits, dtype, B, N, V, row_stride_elems, parent, node_draft_row, M, k,
                            node_token, draft_idx, draft_logit, draft_count, nullptr, 0, draft_temperature, target_temperature,
                            u_accept, u_sample, max_depth, accepted_path, accepted_len, out_token, workspace,
                            workspace_bytes, stream);
}

extern "C" int tslt_tree_verify_packed(int walk, const void* target_logits, int dtype, int B, int N, int V,
                                       long long row_stride_elems, const int* parent, const int* node_draft_row,
                                       int M, int k, const int* node_token, const unsigned int* payload,
                                       int prob_format, float draft_temperature, float target_temperature,
                                       const float* u_accept, const float* u_sample, int max_depth,
                                       int* accepted_path, int* accepted_len, int* out_token, void* workspace,
                                       size_t workspace_bytes, void* stream) {
    if (B > 0 && M > 0 && !payload) return TSLT_ERR_INVALID_ARG;
    static const unsigned int kNoRecords = 0;  // M == 0: nothing is read, but the packed path is still taken
    return tree_verify_impl(walk != 0, target_logits, dtype, B, N, V, row_stride_elems, parent, node_draft_row, M, k,
                            node_token, nullptr, nullptr, nullptr, payload ? payload : &kNoRecords, prob_format,
                            draft_temperature, target_temperature, u_accept, u_sample, max_depth, accepted_path,
                            accepted_len, out_token, workspace, workspace_bytes, stream);
}

#ifdef TSLT_STAMPS
// Timeline build only: the stamps of the last tslt_verify call, [kStampCtas, kStampSlots] nanoseconds
// (resolver CTA of sequence b: slots 0 enter, 1 streaming kernel done, 2 positions judged, 3 draft of the
// stop position loaded, 4 correction token sampled).
extern "C" int tslt_debug_stamps_verify(void* host, size_t bytes) {
    if (bytes > sizeof(unsigned long long) * kStampCtas * kStampSlots) return TSLT_ERR_INVALID_ARG;
    return cudaMemcpyFromSymbol(host, g_stamps, bytes) == cudaSuccess ? TSLT_OK : TSLT_ERR_CUDA;
}
#endif
