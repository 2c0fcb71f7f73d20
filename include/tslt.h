/*
 * tslt.h — C ABI of libtslt: the data-parallel hot path of Truncated Sparse Logits
 * Transmission (TSLT) for distributed speculative decoding, as hand-written CUDA kernels
 * for sm_100a.
 *
 * Conventions shared by every entry point
 *   - plain C ABI, no exceptions; every function returns an int status (TSLT_OK = 0,
 *     negative on error).  Argument errors are found on the host before any launch and
 *     leave the outputs untouched.
 *   - the caller owns every buffer.  Pointers are DEVICE pointers unless marked HOST.  The
 *     library never allocates or frees device memory: scratch comes from a caller-provided
 *     workspace whose size is returned by the matching *_workspace_bytes query.  The
 *     workspace must be 256-byte aligned and must not be shared by calls that can overlap
 *     on the device.
 *   - calls are asynchronous on the caller's stream (a cudaStream_t passed as void*; NULL
 *     is the default stream) and return after enqueueing.
 *   - logits are row-major [rows, V] in fp32 (TSLT_F32) or bf16 (TSLT_BF16); the base
 *     pointer must be 16-byte aligned and row_stride_elems * sizeof(element) must be a
 *     multiple of 16.  -inf logits are legal (probability 0, never selected).  NaN / +inf
 *     logits give unspecified values but never an out-of-bounds access or a hang.  While a
 *     row streams, the exponent z * c (c = log2(e) / T rounded to fp32) is carried in fp32
 *     relative to a reference exponent; every probability that is later formed against the
 *     row's normaliser uses the same rounded c, so a common offset of the logits cancels and
 *     what is left of the rounding (2^-25 relative on c) acts on z minus the row's mean only.
 *     The fp32 product z * c itself is good to 2^-24 relative: lse, mass and the acceptance
 *     probabilities keep their 1e-5 accuracy while |z / T| stays below a few hundred; the
 *     selection (which compares stored logits) is exact whatever their size.
 *   - uniforms are fp32 in [0,1); a value >= 1 is read as the largest float below 1.
 *   - "sample" always means inverse CDF in ascending token index: the first index whose
 *     cumulative mass exceeds u * total.
 *   - kernels of one call hand work over at kernel boundaries; where CTAs of one kernel share a
 *     row (tslt_tree_verify_walk) they meet through a ticket counter in the workspace and the
 *     last one to arrive carries on.  The one wait on another CTA (a row's finish CTA on the
 *     row's streaming CTAs in tslt_sparsify) is one-way and bounded: when it runs out, the CTA
 *     sets TSLT_STATUS_WAIT_FELL_BACK in the status word and waits for the end of the streaming
 *     kernel instead; the results are the same.  The first word of the workspace is that device
 *     status word (0 = nothing to report; every call's first kernel clears it), which
 *     tslt_workspace_status reads back; a non-zero word is reported as TSLT_ERR_DEVICE_STATUS.
 */
#ifndef TSLT_H_
#define TSLT_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TSLT_OK 0
#define TSLT_ERR_INVALID_ARG (-1)
#define TSLT_ERR_UNSUPPORTED (-2)
#define TSLT_ERR_WORKSPACE (-3)
#define TSLT_ERR_CUDA (-4)
#define TSLT_ERR_DEVICE_STATUS (-5)
#define TSLT_ERR_STATIC_SCRATCH (-6)

/* bits of the device status word (tslt_workspace_status) */
#define TSLT_STATUS_WAIT_FELL_BACK 1 /* a bounded device-side wait ran out and took its fall-back; results are valid */
#define TSLT_STATUS_BAD_RECORD 2     /* a packed draft record had a count word outside [0, k]; that row was read as empty */

#define TSLT_F32 0
#define TSLT_BF16 1

/* largest supported k (top-k size, or the candidate cap when top-p is on) */
#define TSLT_MAX_K 1024

/* most vocabulary shards one tslt_sparsify_merge takes; it also needs nshards * k <= 2048 */
#define TSLT_MAX_SHARDS 16

/* size of the scratch array built into the library for tslt_verify_static */
#define TSLT_STATIC_SCRATCH_BYTES (8u << 20)

/* Library version as major * 10000 + minor * 100 + patch. */
int tslt_version(void);

/* Static string for a status code; never NULL. */
const char* tslt_status_string(int status);

/* Synchronous check of the device status word of a workspace used by earlier calls on
 * `stream`: waits for the stream, copies the word back and stores it in *device_status
 * (HOST, nullable).  Returns TSLT_OK if it is zero, TSLT_ERR_DEVICE_STATUS otherwise. */
int tslt_workspace_status(const void* workspace, void* stream, int* device_status);

/* Test and tuning knob, process-wide: how many times (200 ns apart) a finish CTA of tslt_sparsify
 * polls for its row before it records TSLT_STATUS_WAIT_FELL_BACK and waits for the end of the
 * streaming kernel instead.  Default 1 << 22 (about a second); 0 sends every CTA through the
 * fall-back at once.  polls >= 0.  (No counterpart in the paper: it bounds a wait of this
 * implementation.) */
int tslt_set_ready_poll_limit(int polls);

/*
 * Draft side: sparsify-then-sample (Section 3, Solution 1; sampling steps of Algorithms 2
 * and 4).  For each of the B*gamma rows:
 *   q   = softmax(logits / temperature) over the whole vocabulary;
 *   S   = the first n tokens in the order (logit descending, index ascending), where
 *         n = min(k, n*, number of finite logits) and n* is the smallest n whose
 *         cumulative q reaches top_p (the crossing token is kept; top_p >= 1 disables it,
 *         so (k, 1.0) is plain top-k and (cap, rho) is top-rho with a cap);
 *   q~  = q restricted to S and renormalised (the truncation equation of Section 3.1);
 *   num_samples tokens are drawn iid from q~, one uniform each (with replacement).
 * Outputs: idx / logit hold the (token id, stored logit upcast to fp32) pairs of S in
 * ASCENDING token id, padded with -1 / -inf up to k; count = n; token = the samples;
 * lse (nullable) = ln sum exp(logits/temperature); mass (nullable) = sum_{S} q, the
 * retained mass rho of Theorem 1.  A row with no finite logit gives count 0, token -1.
 *
 * Shapes: logits [B*gamma, V] with the given row stride; uniforms, token
 * [B*gamma, num_samples]; idx, logit [B*gamma, k]; count, lse, mass [B*gamma].
 * Requires 1 <= k <= min(V, TSLT_MAX_K), top_p > 0, temperature > 0, num_samples >= 0.
 */
int tslt_sparsify_workspace_bytes(int rows, int V, int k, int num_samples, size_t* bytes);
int tslt_sparsify(const void* logits, int dtype, int B, int gamma, int V,
                  long long row_stride_elems, int k, float top_p, float temperature,
                  int num_samples, const float* uniforms, int* idx, float* logit, int* count,
                  int* token, float* lse, float* mass, void* workspace, size_t workspace_bytes,
                  void* stream);

/*
 * tslt_sparsify over a vocabulary that is split across devices (tensor-parallel output
 * projection): every shard runs the truncation on its own slice, and one small merge turns the
 * shards' results into exactly what tslt_sparsify gives on the whole row.  It rests on two facts:
 * the k best tokens of the row (logit descending, index ascending) are among the k best of
 * their own shards, and the row's normaliser is the sum of the shards' (Section 3.1's truncation
 * equation needs nothing else of the row).
 *
 * tslt_sparsify_shard: tslt_sparsify on the shard's [rows, V_shard] logits with top_p = 1 and no
 * samples.  idx holds indices LOCAL to the shard (ascending, -1 padded), logit the stored logits,
 * count the number kept (min(k, finite logits of the shard)), lse2 [rows] (fp64) the base-2 log of
 * sum 2^(z * log2(e) / temperature) over the shard (-inf if it has no finite logit).  Requires
 * 1 <= k <= min(V_shard, TSLT_MAX_K); workspace as tslt_sparsify_workspace_bytes(rows, V_shard,
 * k, 0) says.
 *
 * tslt_sparsify_merge: part_idx / part_logit [nshards, rows, k], part_count / part_lse2 [nshards,
 * rows] are the shards' outputs side by side in ascending vocabulary order (on several devices:
 * after an all-gather of these 8 k + 12 bytes per shard and row; no logits cross the link);
 * shard_offset is a HOST array of nshards token ids, strictly ascending, the global id of each
 * shard's first logit.  dtype is the element type the shards read (it fixes which logit values
 * can occur).  Outputs, top_p, temperature, num_samples and uniforms as in tslt_sparsify, for the
 * whole-vocabulary row; a part_count outside [0, k] or a part_idx below zero is read as an empty
 * entry.  Requires 1 <= nshards <= TSLT_MAX_SHARDS and nshards * k <= 2048
 * (TSLT_ERR_UNSUPPORTED otherwise); workspace >= 256 bytes (the status word), 256-byte aligned.
 */
int tslt_sparsify_shard(const void* logits, int dtype, int rows, int V_shard,
                        long long row_stride_elems, int k, float temperature, int* idx,
                        float* logit, int* count, double* lse2, void* workspace,
                        size_t workspace_bytes, void* stream);
int tslt_sparsify_merge(int dtype, int rows, int nshards, const int* shard_offset, int k,
                        const int* part_idx, const float* part_logit, const int* part_count,
                        const double* part_lse2, float top_p, float temperature, int num_samples,
                        const float* uniforms, int* idx, float* logit, int* count, int* token,
                        float* lse, float* mass, void* workspace, size_t workspace_bytes,
                        void* stream);

/*
 * Verifier side, single candidate: speculative sampling against the sparse draft
 * (Algorithm 3, with the acceptance ratio p/q~ as in Algorithm 5).  For each sequence b:
 *   p_j = softmax(target_logits[b, j] / target_temperature), j = 0..gamma;
 *   q~_j rebuilt from the received (idx, logit) pairs at draft_temperature;
 *   position j is accepted iff u_accept[b, j] < min(1, p_j(x_j) / q~_j(x_j)), x_j =
 *   draft_token[b, j]; accepted_len[b] = a = number of leading accepted positions;
 *   a < gamma:  out_token[b] ~ norm(max(0, p_a - q~_a)) over the FULL vocabulary;
 *   a = gamma:  out_token[b] ~ p_gamma (the bonus row); both use u_sample[b].
 *   A residual whose total mass is at most 4e-7 (below the accuracy to which p is known; exact
 *   arithmetic gives 0 there, e.g. a draft that equals the target on its support) is taken as
 *   empty and out_token is drawn from the unmodified p_a instead.
 * Optional outputs (nullable): accept_prob[b, j] = min(1, p_j(x_j)/q~_j(x_j)),
 * beta_hat[b, j] = sum_{S_j} min(p_j, q~_j) (the truncated acceptance rate of Section
 * 3.2), lse_p[b, j] = ln sum exp(target row / target_temperature).
 *
 * Shapes: target_logits [B, gamma+1, V]; draft_idx, draft_logit [B, gamma, k] and
 * draft_count [B, gamma] exactly as tslt_sparsify writes them; draft_token, u_accept
 * [B, gamma]; u_sample, accepted_len, out_token [B].  Draft indices outside [0, V) are
 * ignored (probability 0) rather than dereferenced.  Requires gamma < 1024 and
 * V * sizeof(element) <= 4 MiB (TSLT_ERR_UNSUPPORTED otherwise).
 */
int tslt_verify_workspace_bytes(int B, int gamma, int V, int k, size_t* bytes);
int tslt_verify(const void* target_logits, int dtype, int B, int gamma, int V,
                long long row_stride_elems, int k, const int* draft_idx,
                const float* draft_logit, const int* draft_count, const int* draft_token,
                float draft_temperature, float target_temperature, const float* u_accept,
                const float* u_sample, int* accepted_len, int* out_token, float* accept_prob,
                float* beta_hat, float* lse_p, void* workspace, size_t workspace_bytes,
                void* stream);

/*
 * tslt_verify without a workspace argument, for callers that must not allocate device memory.
 * (The paper has no counterpart of this call; it exists for the sake of such callers only.)
 *
 * Who these callers are: a decoding loop inside a serving process that handed every byte of HBM
 * to its own pool at start-up (weights, KV cache) and forbids cudaMalloc afterwards, because
 * cudaMalloc synchronises the whole device and can fail once memory is fragmented or full; or
 * a plug-in written in C whose host framework owns the allocator and gives the plug-in no handle
 * on it.  Such a caller still owns its inputs and outputs and passes them exactly as to
 * tslt_verify; only the scratch (ticket counters and one (max, sum) pair per 2 KB of every target
 * row) comes from the library: a fixed array of TSLT_STATIC_SCRATCH_BYTES (8 MiB) in device
 * memory that every GPU holds from the moment the library is loaded until the process exits.
 *
 *   - Limit: the call is refused with TSLT_ERR_STATIC_SCRATCH, before anything touches the
 *     device, when the scratch tslt_verify would need for these sizes and this dtype exceeds
 *     that size (about B * (gamma + 1) * V * sizeof(element) / 256 bytes; B = 256, gamma = 8,
 *     V = 256000 in bf16 needs 4.6 MiB).  Use tslt_verify with your own workspace for larger
 *     problems.
 *   - The first call on each device looks up the array's device address (the device that is
 *     current at the call); make that first call before any stream capture begins.
 *   - The call itself allocates and frees nothing, on the host or on the device.
 *   - All calls on a device share the one array, which still holds what the previous call wrote;
 *     each call clears the words that must start at zero on its stream before its kernel runs.
 *     Two calls that can overlap on the GPU (different streams, no dependency) race on the array
 *     and give wrong results: serialise them.
 * Arguments, results and every other rule are those of tslt_verify.
 */
int tslt_verify_static(const void* target_logits, int dtype, int B, int gamma, int V,
                       long long row_stride_elems, int k, const int* draft_idx,
                       const float* draft_logit, const int* draft_count, const int* draft_token,
                       float draft_temperature, float target_temperature, const float* u_accept,
                       const float* u_sample, int* accepted_len, int* out_token, float* accept_prob,
                       float* beta_hat, float* lse_p, void* stream);

/*
 * Verifier side, multi-candidate token tree (Algorithm 5 at every node met on the
 * root-to-leaf search of Algorithm 8).  Node 0 is the root (the prefix); parent[i] < i;
 * the children of a node, taken in ascending node id, are its candidates x^(1..k).
 * target_logits[b, n] is the target distribution for the token AFTER node n, so the root
 * row judges the root's children.  Starting at the root with p^(1) = p_node: child c is
 * accepted iff u_accept[b, c] < min(1, p^(i)(x_c) / q~_node(x_c)); on acceptance the walk
 * moves to c; on rejection p^(i+1) = norm(max(0, p^(i) - q~_node)) (after EVERY rejection,
 * duplicates included).  The walk stops at a node whose children were all rejected, where
 * out_token ~ p^(k+1), or at a leaf, where out_token ~ p_leaf; both use
 * u_sample[b, stop node].  accepted_path[b, :] lists the accepted node ids (pad -1) and
 * accepted_len[b] their number.
 *
 * parent and node_draft_row are HOST arrays [N]: node_draft_row[n] is the row (in [0, M))
 * of node n's sparse draft in draft_idx / draft_logit [B, M, k] and draft_count [B, M], or
 * -1 for a leaf.  A node is internal iff it has children iff node_draft_row[n] >= 0.
 * node_token, u_accept, u_sample are [B, N] (entry 0 of node_token / u_accept unused).
 * max_depth >= depth of the tree; accepted_path is [B, max_depth].  N <= 1024.
 */
int tslt_tree_verify_workspace_bytes(int B, int N, int V, int k, size_t* bytes);
int tslt_tree_verify(const void* target_logits, int dtype, int B, int N, int V,
                     long long row_stride_elems, const int* parent, const int* node_draft_row,
                     int M, int k, const int* node_token, const int* draft_idx,
                     const float* draft_logit, const int* draft_count, float draft_temperature,
                     float target_temperature, const float* u_accept, const float* u_sample,
                     int max_depth, int* accepted_path, int* accepted_len, int* out_token,
                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same verification by a root-to-leaf PATH WALK (the "new sequence searching" loop that ends
 * Algorithm 8; Section 4.2): the search only ever uses the nodes on one path, and the uniforms
 * are indexed by node, so verifying just the node each sequence's walk has reached gives the
 * outputs of tslt_tree_verify exactly, while reading at most depth + 1 of the N target rows of a
 * sequence.  One launch per tree level on the caller's stream: the rows of the current nodes are
 * streamed, Algorithm 5 runs at each of them, the walks move to the accepted children; a
 * sequence whose walk has stopped costs nothing in later levels.  Arguments, results and rules
 * are those of tslt_tree_verify; the workspace is smaller (chunk partials of B rows, not B * N)
 * and has its own size query.  Use it when latency or bytes read matter (the rows it skips are
 * never touched); tslt_tree_verify, one streaming pass over all B * N rows, is the form the
 * paper's "in parallel" node loop describes.
 */
int tslt_tree_verify_walk_workspace_bytes(int B, int N, int V, int k, size_t* bytes);
int tslt_tree_verify_walk(const void* target_logits, int dtype, int B, int N, int V,
                          long long row_stride_elems, const int* parent, const int* node_draft_row,
                          int M, int k, const int* node_token, const int* draft_idx,
                          const float* draft_logit, const int* draft_count, float draft_temperature,
                          float target_temperature, const float* u_accept, const float* u_sample,
                          int max_depth, int* accepted_path, int* accepted_len, int* out_token,
                          void* workspace, size_t workspace_bytes, void* stream);

/*
 * Uplink payload (Section 2.2: a transmitted distribution costs entries * (b_prob + b_idx) bits,
 * b_idx = ceil(log2 |V|), b_prob = 32 or 16; Section 3, Solution 1: what is sent are the selected
 * logits and their token ids).  tslt_pack_payload turns the output of tslt_sparsify into what
 * goes over the link, tslt_unpack_payload turns it back into the arrays tslt_verify and
 * tslt_tree_verify take.  The paper fixes the bit widths, not a layout; the layout is:
 *   one record of `words` 32-bit little-endian words per row, `words` given by
 *   tslt_payload_words = 1 + ceil(k * (b_idx + b_prob) / 32); word 0 = n, the row's number of
 *   entries (draft_count); the entries follow as one bit stream, entry e in bits
 *   [e * w, (e + 1) * w), w = b_idx + b_prob, stream bit i being bit (i mod 32) of word
 *   1 + i / 32; inside an entry the low b_idx bits are the token index, the next b_prob bits the
 *   logit's bit pattern in the chosen format.  Bits after the last entry are zero.
 * prob_format: TSLT_PROB_F32 (32 bits, exact), TSLT_PROB_BF16 or TSLT_PROB_F16 (16 bits, the
 * fp32 logit rounded to nearest even; exact whenever the logits came from bf16 storage and the
 * format is bf16).  With a 16-bit format the verifier sees the rounded logits: q~ is the
 * distribution of the rounded values, which is what the draft side must also have sampled from
 * for the method's guarantees to hold exactly; tslt_sparsify samples from the unrounded ones,
 * so with fp32 logits and a 16-bit payload the pair is an approximation (for bf16 logits and a
 * bf16 payload nothing changes).
 * Arguments (device pointers): idx [rows, k] int32 padded with -1, logit [rows, k] fp32 padded
 * with -inf, count [rows] int32 (0 <= count <= k, the first count entries of a row are used),
 * payload [rows, words] uint32.  payload_bits (may be NULL) [rows] int64 gets the paper's
 * figure n * (b_idx + b_prob) per row; the count word is not part of it.  V >= 1, 1 <= k <=
 * TSLT_MAX_K, indices must be in [0, V).  An unpacked count above k (a corrupt record) sets the
 * status flag returned through *device_flag (may be NULL; int32, set to 1, never cleared) and
 * the row is treated as empty.  No workspace.  Errors: TSLT_ERR_INVALID_ARG, TSLT_ERR_UNSUPPORTED
 * (unknown format), TSLT_ERR_CUDA.
 */
#define TSLT_PROB_F32 0
#define TSLT_PROB_BF16 1
#define TSLT_PROB_F16 2
int tslt_payload_words(int k, int V, int prob_format, int* words, int* entry_bits);
int tslt_pack_payload(const int* idx, const float* logit, const int* count, int rows, int k, int V,
                      int prob_format, unsigned int* payload, long long* payload_bits, void* stream);
int tslt_unpack_payload(const unsigned int* payload, int rows, int k, int V, int prob_format,
                        int* idx, float* logit, int* count, int* device_flag, void* stream);

/*
 * The verifiers reading the uplink records directly (Section 3, Solution 1: what arrives at the
 * verifier IS the packed payload; unpacking it to arrays first costs a kernel and a round trip of
 * 8 k bytes per row).  tslt_verify_packed is tslt_verify, and tslt_tree_verify_packed is
 * tslt_tree_verify (walk = 0) or tslt_tree_verify_walk (walk != 0), with `payload` [draft rows,
 * tslt_payload_words(k, V, prob_format)] in place of draft_idx / draft_logit / draft_count: record r
 * is draft row r, exactly as tslt_pack_payload writes it.  Same outputs, workspace sizes and limits
 * as the unpacked calls, bit for bit equal to them on the unpacked arrays.  A record whose count
 * word is outside [0, k] is read as an empty row and sets TSLT_STATUS_BAD_RECORD in the status word.
 */
int tslt_verify_packed(const void* target_logits, int dtype, int B, int gamma, int V,
                       long long row_stride_elems, int k, const unsigned int* payload, int prob_format,
                       const int* draft_token, float draft_temperature, float target_temperature,
                       const float* u_accept, const float* u_sample, int* accepted_len, int* out_token,
                       float* accept_prob, float* beta_hat, float* lse_p, void* workspace,
                       size_t workspace_bytes, void* stream);
int tslt_tree_verify_packed(int walk, const void* target_logits, int dtype, int B, int N, int V,
                            long long row_stride_elems, const int* parent, const int* node_draft_row,
                            int M, int k, const int* node_token, const unsigned int* payload,
                            int prob_format, float draft_temperature, float target_temperature,
                            const float* u_accept, const float* u_sample, int max_depth,
                            int* accepted_path, int* accepted_len, int* out_token, void* workspace,
                            size_t workspace_bytes, void* stream);

/*
 * Truncation diagnostics on pairs of (draft, target) rows: what Section 5's top-K mass and acceptance
 * figures plot, and what Theorem 1 (Section 3.2) and Theorem 2 (Section 4.3) bound.  For row r, with
 * q = softmax(draft_logits[r] / draft_temperature), p = softmax(target_logits[r] / target_temperature):
 *   beta_j[r, j-1]  = beta^(j) = sum_v min(q, p^(j)), the acceptance rate of the j-th candidate, where
 *                     p^(1) = p and p^(j+1) = norm(max(0, p^(j) - q)) (the residual update of Algorithm 5);
 *                     beta^(1) is the acceptance-rate lemma's sum min(q, p) = 1 - TV(q, p);
 *   z_j[r, j-1]     = Z^(j+1) = sum_v max(0, p^(j) - q), the normaliser of that update (= 1 - beta^(j));
 *   theta[r]        = beta^(1) + sum_{i>=2} beta^(i) prod_{j<i} (1 - beta^(j)), the total acceptance;
 *   and for every K = k_list[i] (top-K set of q in the order (logit descending, index ascending),
 *   q^ = q / rho on it and 0 elsewhere: the truncation equation of Section 3.1):
 *   rho[r, i]             = sum over the set of q (sigma = 1 - rho is the truncated mass of Theorem 1),
 *   beta_hat_j[r, i, j-1] = the same chain with q^ in place of q,
 *   theta_hat[r, i]       = its total acceptance.
 * k_list is a HOST array of n_k (1..16) strictly ascending values, each <= min(V, TSLT_MAX_K);
 * 1 <= num_candidates <= 8; a row with fewer finite logits than K uses them all.  The rows are
 * streamed 2 + 2 * num_candidates times: a diagnostic, not a hot path.  Workspace from
 * tslt_diagnostics_workspace_bytes(rows, V, largest K, num_candidates).  All outputs fp32, required.
 */
int tslt_diagnostics_workspace_bytes(int rows, int V, int k_max, int num_candidates, size_t* bytes);
int tslt_diagnostics(const void* draft_logits, const void* target_logits, int dtype, int rows, int V,
                     long long row_stride_elems, const int* k_list, int n_k, int num_candidates,
                     float draft_temperature, float target_temperature, float* beta_j, float* z_j,
                     float* theta, float* rho, float* beta_hat_j, float* theta_hat, void* workspace,
                     size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TSLT_H_ */
