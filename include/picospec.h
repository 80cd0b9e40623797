/*
 * picospec.h -- C-ABI of the B200 (sm_100a) hot path of PicoSpec's separate rejection
 * sampling with sparse compression (arXiv 2603.19133, Sec. 3.3).
 *
 * Conventions for every entry point
 *   - Array arguments are DEVICE pointers owned by the caller unless a comment says "host".
 *     The library never frees or keeps them beyond the asynchronous work it enqueues.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = default
 *     stream).  No entry point synchronises the stream except picospec_status.
 *   - The library allocates device memory only inside picospec_create; the three hot calls
 *     allocate nothing.  A context owns a workspace that the hot calls use as scratch, so
 *     calls on one context must be ordered (one stream at a time); use one context per stream
 *     for concurrent work.
 *   - Logits are row-major with the vocabulary contiguous: element (b, i, v) of a
 *     [B, R, V] tensor lives at base + ((b * R + i) * row_stride_elems + v), R = G for draft
 *     logits and G + 1 for target logits.  row_stride_elems >= V.  Rows whose base address and
 *     pitch are 16-byte aligned take the 128-bit load path; other rows are read element-wise.
 *   - The return value reports errors the host can see (bad arguments, capacity, CUDA launch
 *     errors).  Data errors found by kernels (NaN or +inf logits, a row of -inf only, a
 *     temperature that is not finite and > 0, token / index / count / position out of range)
 *     set bits of a sticky device status word and mark the affected outputs with -1; no kernel
 *     traps or asserts.
 *   - Decisions that floating point takes (accept test, top-p cut, inverse-CDF thresholds) are
 *     taken in fp32-accumulated arithmetic when they are clear of their threshold by more than
 *     the accumulated rounding error, and re-taken in double precision otherwise; the number of
 *     rows that needed the double-precision pass is reported by picospec_status.
 */
#ifndef PICOSPEC_H_
#define PICOSPEC_H_

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define PICOSPEC_API __attribute__((visibility("default")))
#else
#define PICOSPEC_API
#endif

typedef struct picospec_ctx picospec_ctx; /* opaque: workspace, status word, capacities */

typedef enum { PICOSPEC_F32 = 0, PICOSPEC_BF16 = 1 } picospec_dtype;

typedef enum {
    PICOSPEC_OK = 0,
    PICOSPEC_EINVAL = -1,    /* null pointer, negative size, top_p <= 0, unknown dtype ...      */
    PICOSPEC_ECUDA = -2,     /* a CUDA runtime call failed; see picospec_last_cuda_error        */
    PICOSPEC_ECAPACITY = -3, /* B, G, V or k_max exceed what the context was created for        */
    PICOSPEC_EDATA = -4      /* reported by picospec_status only: a kernel found bad data       */
} picospec_err;

/* bits of the device status word */
#define PICOSPEC_ST_TEMPERATURE 1 /* temperature not finite or <= 0                              */
#define PICOSPEC_ST_LOGIT 2       /* NaN or +inf logit, or a row with no finite logit            */
#define PICOSPEC_ST_RANGE 4       /* draft token, sparse index, count or position out of range   */
#define PICOSPEC_ST_INTERNAL 8    /* a bounded wait inside a kernel ran out (outputs not valid)  */

#define PICOSPEC_CHUNK 1024 /* vocabulary entries per level-1 chunk of the residual sampler      */
#define PICOSPEC_MAX_K 1024 /* largest k_max a context accepts                                   */
#define PICOSPEC_MAX_GAMMA 64

/* Create a context on CUDA device `device` able to serve calls with B <= max_batch,
 * G <= max_gamma, V <= max_vocab, k_max <= max_k.  Allocates the workspace (a few MB for the
 * paper's vocabularies).  *out is host memory.  Returns PICOSPEC_OK or an error. */
PICOSPEC_API int picospec_create(picospec_ctx** out, int device, int max_batch, int max_gamma, int max_vocab, int max_k);

/* Free the workspace.  The caller makes sure no enqueued work still uses the context. */
PICOSPEC_API int picospec_destroy(picospec_ctx* ctx);

/* Static, never-freed description of an error code. */
PICOSPEC_API const char* picospec_strerror(int err);

/* cudaError_t of the last failing CUDA call made through this context (0 if none). */
PICOSPEC_API int picospec_last_cuda_error(const picospec_ctx* ctx);

/* The staged kernels wait for their asynchronous copies with a time limit (two seconds by default):
 * a wait that runs out sets PICOSPEC_ST_INTERNAL, the waiting warp stops computing, and the outputs
 * of that call -- and of every later call until the status word is cleared -- are marked invalid
 * (-1); the kernel still waits for every copy it issued before it ends.  This call lowers the limit
 * for later calls on the context (values above two seconds are clamped to it); it exists so that
 * the give-up path can be exercised: with a limit of 0 the first wait that is not already complete
 * gives up.  The paper has no counterpart. */
PICOSPEC_API int picospec_wait_limit(picospec_ctx* ctx, unsigned long long limit_ns);

/* Optional per-kernel timing, for benchmarks.  level 0 = off (default), 1 = bracket the two
 * streaming kernels (one per hot call) with CUDA events on the caller's stream, 2 = bracket every
 * kernel group.  Enabling creates the events (host objects; no device memory) and resets the
 * counters; call it outside timed or captured regions.  The paper has no counterpart. */
#define PICOSPEC_PROF_COMPRESS_STREAM 0  /* compress: streaming filter (or direct select) kernel  */
#define PICOSPEC_PROF_VERIFY_STREAM 1    /* verify / residual_sample: streaming statistics kernel */
#define PICOSPEC_PROF_VERIFY_FINISH 2    /* verify: per-sequence finish kernel                   */
#define PICOSPEC_PROF_VERIFY_PRECISE 3   /* verify: double-precision re-evaluation kernels       */
#define PICOSPEC_PROF_COMPRESS_PRECISE 4 /* compress: double-precision re-evaluation kernels     */
#define PICOSPEC_PROF_COMPRESS_REDO 5    /* compress: direct kernel on rows handed over by the staged one */
#define PICOSPEC_PROF_COMPRESS_FINISH 6  /* compress: per-row sort / cut / emit kernel of the staged path   */
#define PICOSPEC_PROF_KINDS 7
PICOSPEC_API int picospec_profile_enable(picospec_ctx* ctx, int level);

/* Bracket only every `every`-th launch of each kind (default 1 = every launch).  An event between
 * two kernels keeps the second from being scheduled while the first drains, so a benchmark that
 * times whole steps samples the per-kernel brackets sparsely.  every >= 1. */
PICOSPEC_API int picospec_profile_period(picospec_ctx* ctx, int every);

/* Synchronise `cuda_stream`, then return the summed device time (ms, HOST pointer) and the number
 * of launches (HOST pointer) recorded for `kind` since the last read (at most the last 128
 * launches are kept), and reset that counter. */
PICOSPEC_API int picospec_profile_read(picospec_ctx* ctx, int kind, float* total_ms_out, int* launches_out,
                                       void* cuda_stream);

/* The same, launch by launch: the device times (ms) of the launches recorded for `kind` since the
 * last read go to ms_out (HOST array of `capacity` floats), oldest first -- the newest
 * min(capacity, 128) of them -- and their number to *n_out (HOST).  Resets the counter. */
PICOSPEC_API int picospec_profile_samples(picospec_ctx* ctx, int kind, float* ms_out, int capacity, int* n_out,
                                          void* cuda_stream);

/* Synchronise `cuda_stream`, then copy the sticky status word and the cumulative number of rows
 * re-evaluated in double precision to HOST memory (either pointer may be NULL).  If `clear` is
 * non-zero both are reset afterwards.  Returns PICOSPEC_EDATA if the status word is non-zero. */
PICOSPEC_API int picospec_status(picospec_ctx* ctx, int* device_status_out, long long* slow_path_rows_out, int clear,
                    void* cuda_stream);

/* Synchronise `cuda_stream`, then copy two cumulative work counters to HOST memory: out[0] = rows
 * re-evaluated in double precision (the same number picospec_status reports), out[1] = draft rows
 * that the staged compress kernel handed to the direct kernel because their candidates did not
 * fit its buffer (heavy ties, adversarial order, no finite bound).  Both are performance
 * diagnostics; results do not depend on them.  If `clear` is non-zero both are reset.  The paper
 * has no counterpart. */
PICOSPEC_API int picospec_counters(picospec_ctx* ctx, long long* out, int clear, void* cuda_stream);

/* Half 1 -- draft-side sparse compression (Sec. 3.3, Eq. (4): keep the K most probable entries
 * with their vocabulary indices; this library applies it to the drafter's distribution, adds the
 * top-p cut and renormalises).
 *
 * For every row (b, i) of draft_logits [B, G, V]:
 *   q      = softmax(logits / temperature[b])
 *   order  = vocabulary sorted by (logit descending, index ascending)
 *   k_eff  = min(top_k > 0 ? top_k : k_max, k_max, V)
 *   n      = k_eff, or with top_p < 1 the smallest n >= 1 whose first n entries of `order`
 *            reach cumulative probability >= top_p, capped at k_eff
 *   q_idx[b,i,j]  = order[j],  q_prob[b,i,j] = q[order[j]] / sum_{j'<n} q[order[j']]   (j < n)
 *   q_idx[b,i,j]  = -1,        q_prob[b,i,j] = 0                                      (j >= n)
 *   q_count[b,i]  = n
 * If u_draft and draft_tok are non-NULL, draft_tok[b,i] is drawn from the sparse row by inverse
 * CDF in stored order with the uniform u_draft[b,i] in [0,1) (the drafter's own sampling step;
 * the output law of the method is exact only if the candidate comes from this same q~).
 * A row with bad data gets q_count = -1, q_idx = -1, q_prob = 0, draft_tok = -1.
 *
 * temperature [B] fp32 > 0; q_idx, q_prob [B, G, k_max]; q_count [B, G]; u_draft, draft_tok
 * [B, G] or both NULL.  top_k = 0 disables top-k; top_p >= 1 disables top-p; top_p must be > 0.
 */
PICOSPEC_API int picospec_compress(picospec_ctx* ctx, const void* draft_logits, picospec_dtype dtype, int B, int G, int V,
                      long long row_stride_elems, const float* temperature, int top_k, float top_p, int k_max,
                      int* q_idx, float* q_prob, int* q_count, const float* u_draft, int* draft_tok,
                      void* cuda_stream);

/* Half 2a -- target-side verification (Sec. 3.3: the verifier decides each candidate from the
 * probability the drafter gave it; Sec. 2.1: the speculative-sampling accept rule).
 *
 * For every sequence b, with p_i = softmax(target_logits[b, i, :] / temperature[b]), i in [0, G]:
 *   x = draft_tok[b,i];  qx = q_prob of x in sparse row (b,i), 0 if absent
 *   accept_i  = (qx == 0) or u_accept[b,i] < min(1, p_i(x) / qx)
 *   p_draft[b,i]    = p_i(x)
 *   resid_mass[b,i] = sum_v max(0, p_i(v) - q~_i(v))                       (every i < G)
 *   accept_len[b]   = number of leading accepted positions, in [0, G]
 *   *borderline_count = number, over the whole call, of deciding accept tests (every accepted
 *                       one and the first rejected one of each sequence) with
 *                       |p_i(x)/qx - u| <= 1e-6 * u
 * If u_resample and token are non-NULL the call also performs half 2b at position
 * accept_len[b] (residual at a rejected position, p itself at the bonus row G).
 * A sequence with bad data gets accept_len = -1, token = -1, p_draft = resid_mass = -1.
 *
 * target_logits [B, G+1, V]; draft_tok [B, G]; q_idx, q_prob [B, G, k_max]; q_count [B, G];
 * u_accept [B, G] fp32 in [0,1); accept_len [B]; p_draft, resid_mass [B, G] fp32;
 * borderline_count [1] int32; u_resample [B, 2] fp32 in [0,1); token [B].
 */
PICOSPEC_API int picospec_verify(picospec_ctx* ctx, const void* target_logits, picospec_dtype dtype, int B, int G, int V,
                    long long row_stride_elems, const float* temperature, const int* draft_tok, const int* q_idx,
                    const float* q_prob, const int* q_count, int k_max, const float* u_accept, int* accept_len,
                    float* p_draft, float* resid_mass, int* borderline_count, const float* u_resample,
                    int* token, void* cuda_stream);

/* Wire format of sparse rows (Sec. 3.3: the verifier sends K pairs of vocabulary id and
 * probability, under 100 bytes for K = 10, laid out so that the receiver views the arrays in place).  One message, little
 * endian, 4-byte aligned:
 *     0   u32  magic 0x31505350 ("PSP1")
 *     4   u32  R, the number of rows
 *     8   u16  K, the capacity of a dense row
 *     10  u16  probability type: 0 = fp32, 1 = fp16 (round to nearest even)
 *     12  u32  N = sum over rows of max(count, 0)
 *     16  i16  count[R]   (-1 = invalid row), zero-padded to a multiple of 4 bytes
 *     ..  i32  id[N]      rows in order, entries in stored order
 *     ..  prob[N]         fp32 or fp16; the message is zero-padded to a multiple of 4 bytes
 * The id and prob arrays of the message are the receiver's views; picospec_wire_unpack scatters
 * them back into dense [R, K] arrays (padding: id -1, prob 0) for the calls above.
 *
 * picospec_wire_bytes: size of a message (host arithmetic; -1 on bad arguments).
 * picospec_wire_pack: q_idx, q_prob [rows, k], q_count [rows] (device) -> buf (device, 4-byte
 *   aligned, capacity_bytes long).  *bytes_out (DEVICE pointer) = size of the message, or -1 if it
 *   does not fit (then buf holds no message and status bit 4 is set).  A count outside [-1, k]
 *   travels as -1 and sets status bit 4.
 * picospec_wire_unpack: the reverse; a message whose magic, R, K, type, counts or length do not
 *   match is refused as a whole: every row comes back invalid (count -1, id -1, prob 0) and status
 *   bit 4 is set.
 * rows <= max_batch * (max_gamma + 1) of the context, k <= PICOSPEC_MAX_K.
 */
PICOSPEC_API long long picospec_wire_bytes(int rows, long long entries, int prob_type);
PICOSPEC_API int picospec_wire_pack(picospec_ctx* ctx, const int* q_idx, const float* q_prob, const int* q_count, int rows,
                       int k, int prob_type, void* buf, long long capacity_bytes, long long* bytes_out,
                       void* cuda_stream);
PICOSPEC_API int picospec_wire_unpack(picospec_ctx* ctx, const void* buf, long long bytes, int rows, int k, int* q_idx,
                         float* q_prob, int* q_count, void* cuda_stream);

/* Half 2a on rows as they arrive -- incremental verification (Sec. 3.2: the verifier works on a
 * prefix of the segment while the drafter is still producing the rest; Sec. 3.3: latency-aware
 * truncation makes the number of drafted tokens differ between sequences).
 *
 * One call handles the target rows [r0, r1) of every sequence that is still undecided and never
 * reads a row outside that range; a chain of calls over consecutive ranges that together cover
 * [0, G + 1), each passing the previous call's state_out as state_in, gives every sequence the
 * accept_len and token picospec_verify gives it.
 *   gamma[b] (NULL: G) = drafted tokens of sequence b, in [0, G]; its rows are 0 .. gamma[b], the
 *                        last one the bonus row; rows beyond it are never read.
 *   state_in[b] (NULL: all 1): 1 = every position before r0 was accepted; 0 = decided by an
 *                        earlier call: the sequence is skipped, of its outputs only
 *                        state_out[b] = 0 is written.
 * For an undecided sequence the positions i in [r0, min(r1, gamma)) get the accept test of
 * picospec_verify, with p_draft[b,i] and resid_mass[b,i] written for exactly those positions.
 *   first rejection at i:                       accept_len = i, token from the residual of row i
 *   all accepted and r0 <= gamma < r1:          accept_len = gamma, token from p at row gamma
 *   otherwise (undecided):                      accept_len = -2, token = -2, state_out = 1
 * Decided sequences get state_out = 0.  *borderline_count counts this call's deciding tests.
 * Bad data inside the range, gamma[b] outside [0, G], or gamma[b] < r0 for an undecided
 * sequence: accept_len = -1, token = -1, state_out = 0, the range's p_draft = resid_mass = -1,
 * and the matching status bit.
 *
 * 0 <= r0 < r1 <= G + 1, else PICOSPEC_EINVAL.  gamma, state_in [B] int32 or NULL; state_out [B]
 * int32; every other array as in picospec_verify.  state_in and state_out may be the same
 * array.
 */
PICOSPEC_API int picospec_verify_range(picospec_ctx* ctx, const void* target_logits, picospec_dtype dtype, int B, int G,
                          int V, long long row_stride_elems, const float* temperature, const int* gamma, int r0,
                          int r1, const int* state_in, const int* draft_tok, const int* q_idx, const float* q_prob,
                          const int* q_count, int k_max, const float* u_accept, int* accept_len, float* p_draft,
                          float* resid_mass, int* borderline_count, const float* u_resample, int* token,
                          int* state_out, void* cuda_stream);

/* Half 2b -- local resampling (Sec. 3.3: the corrected token is drawn from
 * norm(max(0, P_j(x) - Q_j(x)))).
 *
 * For every sequence b, row j = pos[b] of its target logits: weights r_v = max(0, p_j(v) - q~_j(v))
 * if j < G and the sparse row (b, j) is non-empty, else r_v = p_j(v) (bonus row; also the
 * fallback when the residual vanishes, where Sec. 3.3's norm() is undefined: a residual whose
 * total mass is at most 1e-12 of the row's counts as vanished, because the chunk masses are
 * differences of double-precision sums).  The token is drawn by a two-level inverse
 * CDF with chunks of PICOSPEC_CHUNK vocabulary entries: u_resample[b,0] picks the first chunk c
 * whose cumulative mass exceeds u0 * sum(r); u_resample[b,1] picks the first entry of that chunk
 * whose cumulative weight inside the chunk exceeds u1 * mass(c).  Entries of zero weight are
 * never drawn.  mass[b] (optional) = sum_v r_v.
 *
 * pos [B] in [0, G]; other arrays as in picospec_verify; token [B]; mass [B] fp32 or NULL.
 */
PICOSPEC_API int picospec_residual_sample(picospec_ctx* ctx, const void* target_logits, picospec_dtype dtype, int B, int G,
                             int V, long long row_stride_elems, const float* temperature, const int* pos,
                             const int* q_idx, const float* q_prob, const int* q_count, int k_max,
                             const float* u_resample, int* token, float* mass, void* cuda_stream);

/* The paper's own data flow, verifier side -- Sec. 3.3, Eq. (4): of the target distribution at the
 * rejected position the verifier keeps the K most probable components, each with its vocabulary
 * index, and sends only those.
 *
 * For every sequence b, row j = pos[b] of target_logits [B, R, V] (R rows per sequence):
 *   p      = softmax(logits / temperature[b])
 *   order  = vocabulary sorted by (logit descending, index ascending)
 *   p_idx[b,t] = order[t], p_prob[b,t] = p[order[t]] for t < n = min(k, V)  (NOT renormalised: the
 *                paper sends the components as they are); -1 and 0 beyond n; p_count[b] = n
 * A sequence with bad data (temperature, position outside [0, R), NaN / +inf logits) gets
 * p_count = -1, p_idx = -1, p_prob = 0 and sets the status word.
 * The usual verifier call before it is picospec_verify with one-entry sparse rows holding the
 * drafted token and the scalar q(x) the edge sent (k_max = 1), without the fused sample.
 *
 * pos [B] int32 in [0, R); p_idx, p_prob [B, k]; p_count [B]; k <= the context's max_k, R - 1 <= its
 * max_gamma. */
PICOSPEC_API int picospec_target_topk(picospec_ctx* ctx, const void* target_logits, picospec_dtype dtype, int B, int R,
                         int V, long long row_stride_elems, const float* temperature, const int* pos, int k,
                         int* p_idx, float* p_prob, int* p_count, void* cuda_stream);

/* The paper's own data flow, edge side -- Sec. 3.3: the edge draws the corrected token by itself,
 * from the normalised positive part of (received target components - its own draft distribution).
 *
 * For every sequence b, with Q = softmax(draft_logits[b, pos[b], :] / temperature[b]) (the edge's own
 * dense row) and the transmitted components (p_idx, p_prob, p_count) of the target distribution
 * (a component that was not transmitted counts as zero, so only transmitted indices can be drawn):
 *   r_t = max(0, p_prob[b,t] - Q(p_idx[b,t])),  R = sum_t r_t                      (stored order)
 *   token[b] = p_idx[b, first t whose running sum of r exceeds u[b] * R]  (else the last t with r_t > 0)
 *   if R = 0 (Q covers every transmitted component) the draw is from p_prob itself
 *   mass[b] (optional) = the total of the weights drawn from
 * Bad data (temperature, position, count or index out of range, NaN / +inf logits): token = -1,
 * mass = -1, status word set.  Unlike picospec_residual_sample this is not an exact sampler of the
 * true residual unless every component was transmitted (k >= V): it is the truncation the paper
 * proposes.
 *
 * draft_logits [B, R, V]; pos [B] in [0, R); p_idx, p_prob [B, k]; p_count [B] in [1, k];
 * u [B] fp32 in [0,1); token [B]; mass [B] fp32 or NULL. */
PICOSPEC_API int picospec_edge_resample(picospec_ctx* ctx, const void* draft_logits, picospec_dtype dtype, int B, int R,
                           int V, long long row_stride_elems, const float* temperature, const int* pos,
                           const int* p_idx, const float* p_prob, const int* p_count, int k, const float* u,
                           int* token, float* mass, void* cuda_stream);

/* Vocabulary-parallel verification -- Sec. 4.1: the verifier model runs on two to four GPUs, so its
 * output layer leaves the target logits sharded along the vocabulary.  Rank r of `ranks` holds the
 * columns [v0, v0 + Vs) of every row of target_logits [B, G+1, V]: v0 = r * chunks_per_rank *
 * PICOSPEC_CHUNK, every rank but the last holds chunks_per_rank chunks, the last one the rest.  One
 * verification is the sequence below, the same on every rank; the two kinds of exchange between the
 * steps are the caller's (an all-gather and an element-wise maximum over ranks, e.g. NCCL), the
 * library never touches another rank's memory.  Results equal picospec_verify on the whole rows.
 *
 *   picospec_vp_local    own slice -> records_local [B*(G+1), chunks_per_rank, 2] fp32 (per chunk: largest
 *                        logit, sum of 2^((l - max) log2(e)/T)) and entries_local [B*G, k_max+1] fp32 (the
 *                        slice's logits at the stored entries, last slot: at the drafted token; -inf where
 *                        the slice does not hold the index)
 *   exchange             records_all [ranks, B*(G+1), chunks_per_rank, 2] = all-gather(records_local);
 *                        entries_all = max over ranks(entries_local)
 *   picospec_vp_decide   (sums_all = NULL) accept tests, p_draft, resid_mass, accept_len, borderline count
 *                        as in picospec_verify, and pick [B,4] int32: sampled row, picked chunk, flags, rows
 *   picospec_vp_draw     (sums_all = NULL) the owner of a picked chunk draws the token inside it from its
 *                        slice -> tok_flag_local [2, B] int32: token or -1; 1 if too close to call
 *   exchange             tok_flag_all = max over ranks(tok_flag_local)
 *   picospec_vp_queue    token [B] <- tok_flag_all; the context's list of sequences for the
 *                        double-precision pass (the same on every rank)
 *   picospec_vp_exact    own slice -> sums_local [B*(G+1), chunks_per_rank] fp64: exact chunk sums of the
 *                        listed sequences' rows (other entries are not written)
 *   exchange             sums_all [ranks, B*(G+1), chunks_per_rank] = all-gather(sums_local)
 *   picospec_vp_decide   (sums_all given) the listed sequences again, in double precision
 *   picospec_vp_draw     (sums_all given) their draws -> tok_flag_local
 *   exchange             tok_flag_all = max over ranks(tok_flag_local)
 *   picospec_vp_merge    token [B] <- the redone tokens
 * All calls of one verification use one context and one stream.  All arrays are device pointers;
 * capacity and data errors are reported as for picospec_verify. */
PICOSPEC_API int picospec_vp_local(picospec_ctx* ctx, const void* slice_logits, picospec_dtype dtype, int B, int G, int Vs,
                                   int v0, long long row_stride_elems, int chunks_per_rank, const float* temperature,
                                   const int* draft_tok, const int* q_idx, const int* q_count, int k_max,
                                   float* records_local, float* entries_local, void* cuda_stream);
PICOSPEC_API int picospec_vp_decide(picospec_ctx* ctx, int B, int G, int V, int ranks, int chunks_per_rank,
                                    const float* records_all, const double* sums_all, const float* entries_all,
                                    const float* temperature, const int* draft_tok, const int* q_idx,
                                    const float* q_prob, const int* q_count, int k_max, const float* u_accept,
                                    const float* u_resample, int* accept_len, float* p_draft, float* resid_mass,
                                    int* borderline_count, int* pick, void* cuda_stream);
PICOSPEC_API int picospec_vp_draw(picospec_ctx* ctx, const void* slice_logits, picospec_dtype dtype, int B, int G, int V,
                                  int v0, long long row_stride_elems, int rank, int ranks, int chunks_per_rank,
                                  const float* records_all, const double* sums_all, const float* temperature,
                                  const int* q_idx, const float* q_prob, const int* q_count, int k_max,
                                  const float* u_resample, const int* pick, int* tok_flag_local, void* cuda_stream);
PICOSPEC_API int picospec_vp_queue(picospec_ctx* ctx, int B, int G, const int* pick, const int* tok_flag_all, int* token,
                                   void* cuda_stream);
PICOSPEC_API int picospec_vp_exact(picospec_ctx* ctx, const void* slice_logits, picospec_dtype dtype, int B, int G, int Vs,
                                   long long row_stride_elems, int chunks_per_rank, const float* temperature,
                                   double* sums_local, void* cuda_stream);
PICOSPEC_API int picospec_vp_merge(picospec_ctx* ctx, int B, const int* tok_flag_all, int* token, void* cuda_stream);

/* Verification without any allocation -- the paper has no counterpart; this entry point exists
 * for callers that cannot obtain device memory at all.  Two kinds of caller are meant: a plugin
 * inside a serving engine that has already claimed the whole of the GPU's memory for its own
 * pools (cudaMalloc fails there, and so would picospec_create, which allocates the workspace),
 * and a latency-critical loop that must not take the device-wide synchronisation cudaMalloc and
 * cudaFree imply.  Such callers pass their own input and output buffers as usual and need no
 * context.
 *
 * Same computation, arguments and outputs as picospec_verify (including the fused half 2b when
 * u_resample and token are non-NULL), minus the context.  The workspace the kernels need between
 * their passes lives in a fixed array inside the library's device image (about 1 MB, held by
 * every GPU that loads the library until the process exits), so the problem must fit it:
 *     B * (G + 1) <= PICOSPEC_STATIC_MAX_ROWS   and   V <= PICOSPEC_STATIC_MAX_VOCAB
 * (k_max <= PICOSPEC_MAX_K, G <= PICOSPEC_MAX_GAMMA as everywhere); anything larger is rejected
 * with PICOSPEC_ECAPACITY before any work is enqueued.
 *
 * device_status_out (DEVICE pointer to one int, or NULL) receives this call's status bits
 * (PICOSPEC_ST_*) once the enqueued work has run; slow_rows_out (DEVICE pointer to one
 * long long, or NULL) the number of rows this call re-evaluated in double precision.
 *
 * The call makes no cudaMalloc / cudaFree and calls nothing that allocates.  Its first use on a
 * device looks up the address of the fixed array for that device (a host-side query, done once
 * per device with that device current); make that first call outside any stream capture.
 * Every call on a device shares the one array and the array keeps what the previous call left
 * in it; the call clears the few words that must start at zero itself.  Two calls whose work
 * overlaps on the GPU (different streams, or several host threads) race on the array: order
 * them on one stream. */
#define PICOSPEC_STATIC_MAX_ROWS 256
#define PICOSPEC_STATIC_MAX_VOCAB 262144
PICOSPEC_API int picospec_verify_static(const void* target_logits, picospec_dtype dtype, int B, int G, int V,
                           long long row_stride_elems, const float* temperature, const int* draft_tok,
                           const int* q_idx, const float* q_prob, const int* q_count, int k_max,
                           const float* u_accept, int* accept_len, float* p_draft, float* resid_mass,
                           int* borderline_count, const float* u_resample, int* token,
                           int* device_status_out, long long* slow_rows_out, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* PICOSPEC_H_ */
