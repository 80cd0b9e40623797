// Target-side kernels: streaming chunk statistics, per-sequence finish (accept test, scan,
// residual mass, two-level sampler) and the double-precision re-evaluation of flagged sequences.
#pragma once
#include "common.cuh"
#include "precise_kernels.cuh"
#include "stream_pipeline.cuh"

namespace picospec {

struct VerifyArgs {
    const void* logits;        // target logits [B, G+1, V]
    long long row_stride;      // elements
    int B, G, V, nch, k_max;
    int sample_only;           // 1: residual_sample entry point (row pos[b] only)
    // incremental verification: only the target rows [r0, r1) are read, for sequences that are
    // still undecided; the whole batch at once is r0 = 0, r1 = G + 1 with the pointers null
    int r0 = 0, r1 = -1;
    const int* gamma = nullptr;     // [B] drafted tokens per sequence (rows 0 .. gamma[b]); null: G
    const int* state_in = nullptr;  // [B] 1 = undecided so far, 0 = decided earlier (skipped); null: all 1
    int* state_out = nullptr;       // [B] or null
    const float* temperature;  // [B]
    const int* draft_tok;      // [B,G]
    const int* q_idx;          // [B,G,k_max]
    const float* q_prob;
    const int* q_count;        // [B,G]
    const float* u_accept;     // [B,G]
    const int* pos;            // [B] (sample_only)
    const float* u_resample;   // [B,2] or null
    int* accept_len;           // [B]
    float* p_draft;            // [B,G]
    float* resid_mass;         // [B,G]
    int* borderline;           // [1]
    int* token;                // [B] or null
    float* mass;               // [B] or null (sample_only)
    // Vocabulary-parallel verification (the logits are sharded along the vocabulary over several
    // ranks): the chunk records of all ranks lie rank after rank, [ranks, rows, chunks_per_rank], and
    // chunk c of the vocabulary is record c % chunks_per_rank of rank c / chunks_per_rank; one rank,
    // chunks_per_rank = nch is the plain layout.  entry_logits, if set, holds the target logits at the
    // stored entries (slots 0 .. k_max - 1) and at the drafted token (slot k_max) of every draft
    // position, gathered from the ranks that own them: the finish kernel then reads no logits itself
    // and hands the draw inside the picked chunk to that chunk's owner through `pick`.
    int chunks_per_rank = 0;        // 0: nch
    long long rank_stride = 0;      // records between two ranks' blocks
    int stats_pitch = 0;            // records per row written by the streaming pass (0: nch)
    const float* entry_logits = nullptr;   // [B*G, k_max + 1]
    int* pick = nullptr;            // [B, 4]: sampled row, picked chunk (-1: none), flags, unused
    // workspace
    float2* stats;             // [B*(G+1), nch]: (chunk max logit, sum of 2^(l*c32 - max*c32))
    float* row_max;            // [B*(G+1)]
    double* dsum;              // [B*(G+1), nch]: exact chunk sums of flagged sequences
    int* queue;                // [B] flagged sequences
    unsigned long long* need_rows;  // [B] per flagged sequence: bit i = row i needs exact chunk sums
    int* queue_count;          // [1]
    int* rowq;                 // [B*(G+1)] rows (of the logits tensor) whose exact chunk sums are wanted
    int* rowq_count;           // [1]
    unsigned* status;          // sticky status word
    unsigned long long* slow_rows;  // cumulative rows re-evaluated in double precision
};

// ---------------------------------------------------------------------------------------------
// Streaming pass, direct variant (rows that are not 16-byte aligned): one warp per 1024-entry
// chunk, read straight from global memory and software-pipelined over two register buffers.
// Per chunk: exact maximum logit and the fp32 sum of 2^((l - max) * log2e / T).
// ---------------------------------------------------------------------------------------------
// one (row, chunk) item of the direct variant
template <typename T> struct ItemMeta {
    const T* row;
    int v0;
    float c32;
    long long slot;  // index into stats
    bool valid;
};

// Row r of the rows a verify call streams -> (sequence, row of the logits tensor); false: the row
// is not read (sequence decided earlier, or the row lies beyond the sequence's bonus row).
__device__ __forceinline__ bool streamed_row(const VerifyArgs& a, int r, int& b, int& src_row) {
    const int nr = a.r1 - a.r0;
    b = r / nr;
    const int i = a.r0 + (r - b * nr);
    src_row = b * (a.G + 1) + i;
    if (a.state_in && a.state_in[b] == 0) return false;
    if (a.gamma && i > a.gamma[b]) return false;
    return true;
}

// index of the record of (row, chunk c of the vocabulary) in stats / dsum
__device__ __forceinline__ long long record_index(const VerifyArgs& a, int row, int c) {
    if (a.chunks_per_rank == 0) return (long long)row * a.nch + c;      // one rank: the plain layout
    const int L = a.chunks_per_rank;
    const int r = c / L;
    return (long long)r * a.rank_stride + (long long)row * L + (c - r * L);
}
// flags of VerifyArgs::pick
constexpr int PICK_RESIDUAL = 1, PICK_FLAGGED = 2, PICK_DRAW_ONLY = 4, PICK_MASS_ONLY = 8;

template <typename T> __device__ __forceinline__ ItemMeta<T> decode_item(const VerifyArgs& a, long long item) {
    ItemMeta<T> m;
    const int r = (int)(item / a.nch);
    const int c = (int)(item - (long long)r * a.nch);
    int b, src_row;
    m.valid = true;
    if (a.sample_only) {
        b = r;
        const int j = a.pos[b];
        if (j < 0 || j > a.G) m.valid = false;
        src_row = b * (a.G + 1) + (m.valid ? j : 0);
    } else {
        if (!streamed_row(a, r, b, src_row)) m.valid = false;
    }
    const float Tb = a.temperature[b];
    if (!temp_ok(Tb)) m.valid = false;
    m.c32 = temp_scale(Tb);
    m.row = reinterpret_cast<const T*>(a.logits) + (long long)src_row * a.row_stride;
    m.v0 = c * CHUNK;
    m.slot = (long long)src_row * (a.stats_pitch > 0 ? a.stats_pitch : a.nch) + c;
    return m;
}

template <typename T> __device__ __forceinline__ void chunk_stats_compute(const ChunkRegs<T>& regs, const ItemMeta<T>& m,
                                                                          float2* stats, int lane) {
    const float lm = regs.lane_max();
    // NaN anywhere in the chunk: the exp-sum below turns NaN and the finish kernel reports it
    const float cm = warp_max(lm);
    const float off = __fmul_rn(cm, m.c32);
    float s = 0.f;
    if (cm > -CUDART_INF_F) s = lane_exp_sum(regs, m.c32, off);
    if (lm != lm) s = CUDART_NAN_F;
    s = warp_sum(s);
    if (lane == 0) stats[m.slot] = make_float2(cm, s);
}

template <typename T, bool ALIGNED>
__global__ void __launch_bounds__(THREADS, 4) chunk_stats_kernel(VerifyArgs a) {
    grid_dependency_sync();
    const int lane = threadIdx.x & 31;
    const long long gw = (long long)blockIdx.x * WARPS + (threadIdx.x >> 5);
    const long long nw = (long long)gridDim.x * WARPS;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        *a.queue_count = 0;
        *a.rowq_count = 0;
        if (a.borderline) *a.borderline = 0;
    }
    const long long total = (long long)(a.sample_only ? a.B : a.B * (a.r1 - a.r0)) * a.nch;
    long long itA = gw;
    if (itA >= total) return;
    ChunkRegs<T> A, Bf;
    ItemMeta<T> mA = decode_item<T>(a, itA), mB;
    if (mA.valid) A.template load<ALIGNED>(mA.row, mA.v0, a.V, lane);
    for (;;) {
        const long long itB = itA + nw;
        const bool hasB = itB < total;
        if (hasB) {
            mB = decode_item<T>(a, itB);
            if (mB.valid) Bf.template load<ALIGNED>(mB.row, mB.v0, a.V, lane);
        }
        if (mA.valid) chunk_stats_compute<T>(A, mA, a.stats, lane);
        if (!hasB) break;
        itA = itB + nw;
        const bool hasA = itA < total;
        if (hasA) {
            mA = decode_item<T>(a, itA);
            if (mA.valid) A.template load<ALIGNED>(mA.row, mA.v0, a.V, lane);
        }
        if (mB.valid) chunk_stats_compute<T>(Bf, mB, a.stats, lane);
        if (!hasA) break;
    }
}

// ---------------------------------------------------------------------------------------------
// Streaming pass through shared memory (rows whose base, pitch and length are multiples of 16
// bytes).  A tile is TILE_CHUNKS consecutive chunks of one row; CTA c takes tiles c, c + grid,
// c + 2 grid, ...  Warp 8 lane 0 is the producer: it keeps STAGES bulk copies in flight.  Each of
// the 8 consumer warps moves its chunk of a landed tile to registers, hands the stage back and
// then reduces the chunk to (maximum logit, fp32 sum of 2^((l - max) * log2e / T)).
// ---------------------------------------------------------------------------------------------
struct TileDesc {
    int src_row;   // row of the logits tensor
    int c0;        // first chunk of the tile
    float c32;     // log2(e) / T of the row's sequence
    int valid;     // 0: bad temperature or position, or a row that is not read: nothing was copied
};

template <typename T>
__global__ void __launch_bounds__(STREAM_THREADS, StreamCfg<T>::CTAS_PER_SM) chunk_stats_bulk_kernel(VerifyArgs a, int tiles_per_row,
                                                                             long long total_tiles,
                                                                             unsigned long long wait_limit_ns) {
    extern __shared__ __align__(1024) unsigned char stage_mem[];
    constexpr int STAGES = StreamCfg<T>::STAGES;
    constexpr int CPW = StreamCfg<T>::CPW;
    constexpr int TCH = TileGeom<T>::CHUNKS;
    constexpr int TILE_BYTES = TileGeom<T>::TILE_BYTES;
    __shared__ __align__(8) uint64_t full[STAGES], empty[STAGES];
    __shared__ TileDesc desc[STAGES];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], WARPS);
        }
        mbar_init_fence();
    }
    grid_dependency_sync();
    if (tid == 0 && blockIdx.x == 0) {
        *a.queue_count = 0;
        *a.rowq_count = 0;
        if (a.borderline) *a.borderline = 0;
    }
    __syncthreads();

    if (warp == WARPS) {
        // ---- producer ---------------------------------------------------------------------
        if (lane != 0) return;
        const uint64_t pol = l2_evict_first_policy();
        long long t = blockIdx.x;
        for (uint32_t i = 0; t < total_tiles; ++i, t += gridDim.x) {
            const int s = (int)(i % STAGES);
            const uint32_t round = i / STAGES;
            if (round > 0) {
                const int wr = mbar_wait_twice(&empty[s], (round - 1) & 1, wait_limit_ns);
                if (wr != WAIT_OK) atomicOr(a.status, ST_INTERNAL);
                if (wr == WAIT_LOST) break;       // nothing more is issued
            }
            const int r = (int)(t / tiles_per_row);
            const int tc = (int)(t - (long long)r * tiles_per_row);
            TileDesc d;
            d.valid = 1;
            int b;
            if (a.sample_only) {
                b = r;
                const int j = a.pos[b];
                if (j < 0 || j > a.G) d.valid = 0;
                d.src_row = b * (a.G + 1) + (d.valid ? j : 0);
            } else {
                if (!streamed_row(a, r, b, d.src_row)) d.valid = 0;
            }
            const float Tb = a.temperature[b];
            if (!temp_ok(Tb)) d.valid = 0;
            d.c32 = temp_scale(Tb);
            d.c0 = tc * TCH;
            desc[s] = d;
            if (d.valid) {
                const int v0 = d.c0 * CHUNK;
                const int v1 = min(a.V, v0 + TCH * CHUNK);
                const uint32_t bytes = (uint32_t)(v1 - v0) * (uint32_t)sizeof(T);
                const T* src = reinterpret_cast<const T*>(a.logits) + (long long)d.src_row * a.row_stride + v0;
                mbar_arrive_expect_tx(&full[s], bytes);
                bulk_load(stage_mem + s * TILE_BYTES, src, bytes, &full[s], pol);
            } else {
                mbar_arrive(&full[s]);
            }
        }
        return;
    }

    // ---- consumers ------------------------------------------------------------------------
    long long t = blockIdx.x;
    bool late = false;      // a wait ran out: this warp computes no more, but keeps taking tiles
    for (uint32_t i = 0; t < total_tiles; ++i, t += gridDim.x) {
        const int s = (int)(i % STAGES);
        const uint32_t round = i / STAGES;
        const int wr = mbar_wait_twice(&full[s], round & 1, wait_limit_ns);
        if (wr != WAIT_OK) {
            late = true;
            if (lane == 0) atomicOr(a.status, ST_INTERNAL);
            if (wr == WAIT_LOST) break;
        }
        const TileDesc d = desc[s];
#pragma unroll
        for (int q = 0; q < CPW; ++q) {
            const int c = d.c0 + warp * CPW + q;
            const bool work = d.valid && c < a.nch && !late;
            ChunkRegs<T> regs;
            if (work) load_staged(regs, stage_mem + s * TILE_BYTES + (warp * CPW + q) * (CHUNK * (int)sizeof(T)), c * CHUNK, a.V, lane);
            if (q == CPW - 1) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[s]);     // the warp's chunks are in registers or done
            }
            if (work) {
                // chunk maximum with NaN ignored; a NaN (or +inf) logit turns the exp-sum into NaN by
                // itself, which the finish kernel reports; a chunk of -inf only sums to zero
                const float cm = warp_max_redux(regs.lane_max_plain());
                const float off = cm > -CUDART_INF_F ? __fmul_rn(cm, d.c32) : 0.f;
                const float sum = warp_sum(lane_exp_sum2(regs, d.c32, off));
                if (lane == 0) a.stats[(long long)d.src_row * (a.stats_pitch > 0 ? a.stats_pitch : a.nch) + c] = make_float2(cm, sum);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Finish: one CTA per sequence.
// ---------------------------------------------------------------------------------------------
struct FinishShared {
    double Z[MAX_G1];     // normaliser on the scale of Weight<>
    double Zraw[MAX_G1];  // the same sum on the streaming pass's own scale (fast path)
    float mx[MAX_G1];
    int bad;
    int acc[MAX_G1], amb[MAX_G1], bord[MAX_G1], small[MAX_G1];
    double warp_tot[WARPS];
    double red[WARPS];
    int tok, last, flag;
    int cstar;
    double Rtot;
    float qloc[CHUNK];
};

// queue entries of the verify path: the sequence, plus a flag
constexpr int QUEUE_SEQ_MASK = 0x1FFFFFFF, QUEUE_DRAW_ONLY = 0x40000000, QUEUE_MASS_ONLY = 0x20000000;

// bit i of a sequence's row mask (rows beyond 63 always count as set)
__device__ __forceinline__ bool row_needed(unsigned long long need, int i) { return i >= 64 || ((need >> i) & 1ull); }

template <typename T>
__device__ __forceinline__ void row_stats(const VerifyArgs& a, int src_row, float c32, int lane, bool exact, double& Z,
                                          double& Zraw, float& mx, bool& bad) {
    // combine the chunk statistics of one row (called by a full warp): the exact double-precision
    // chunk sums if they were recomputed for this row, else the fp32 streaming statistics
    bad = false;
    Zraw = 0.0;
    if (exact) {
        mx = a.row_max[src_row];
        double s = 0.0;
        for (int c = lane; c < a.nch; c += 32) s += a.dsum[record_index(a, src_row, c)];
        Z = warp_sum(s);
    } else {
        const float2* st = a.stats;
        float m = -CUDART_INF_F;
        bool nan = false;
        for (int c = lane; c < a.nch; c += 32) {
            float2 v = st[record_index(a, src_row, c)];
            m = fmaxf(m, v.x);
            nan |= (v.y != v.y);
        }
        m = warp_max(m);
        nan = __any_sync(0xffffffffu, nan);
        mx = m;
        bad = nan || !(m > -CUDART_INF_F) || !(m < CUDART_INF_F);
        double s = 0.0;
        if (!bad) {
            const double off = (double)__fmul_rn(m, c32);
            for (int c = lane; c < a.nch; c += 32) {
                float2 v = st[record_index(a, src_row, c)];
                if (v.x > -CUDART_INF_F) s += (double)v.y * exp2((double)__fmul_rn(v.x, c32) - off);
            }
        }
        Zraw = warp_sum(s);
        if (!(Zraw > 0.0)) bad = true;
        Z = bad ? 0.0 : Zraw * stream_sum_scale(m, c32);
    }
}

// Level 2 of the sampler, by the 256 threads of a CTA: the token inside chunk `cs` of a row whose
// logits start at `row` with vocabulary index `vbase` (0 for a whole row; the first index of the
// slice when the vocabulary is sharded).  Weights are max(0, p - q~) with the stored entries
// (idx, prob)[0 .. n) if use_resid, else p.  Sets sh.flag when the fast pass cannot call the draw.
template <typename T, bool PRECISE>
__device__ __forceinline__ int level2_draw(const VerifyArgs& a, const T* row, int vbase, int cs, const int* idx,
                                           const float* prob, int n, bool use_resid, const Weight<PRECISE>& wt,
                                           double invZ, float u2, FinishShared& sh) {
    const int tid = threadIdx.x;
    // the 1024 entries of chunk cs, four consecutive entries per thread
    const int v0 = cs * CHUNK;
    for (int k = tid; k < CHUNK; k += THREADS) sh.qloc[k] = 0.f;
    if (tid == 0) {
        sh.tok = 0x7fffffff;
        sh.last = -1;
    }
    __syncthreads();
    if (use_resid)
        for (int k = tid; k < n; k += THREADS) {
            const int v = idx[k];
            if (v >= v0 && v < v0 + CHUNK) sh.qloc[v - v0] = prob[k];
        }
    __syncthreads();
    double r[4], cum[4], qsum = 0.0, loc = 0.0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int v = v0 + tid * 4 + e;
        double w = 0.0;
        if (v < a.V) w = wt(load_logit(row, v - vbase)) * invZ;
        const double q = (double)sh.qloc[tid * 4 + e];
        qsum += q;
        double d = w - q;
        r[e] = d > 0.0 ? d : 0.0;
        loc += r[e];
        cum[e] = loc;
    }
    double M;
    const double incl = block_scan_incl(loc, sh.warp_tot, M);
    const double base = incl - loc;
    double Q;
    block_scan_incl(qsum, sh.warp_tot, Q);
    const double thr2 = (double)u2 * M;
    int mine = 0x7fffffff, mylast = -1;
#pragma unroll
    for (int e = 3; e >= 0; --e) {
        if (base + cum[e] > thr2) mine = v0 + tid * 4 + e;
        if (r[e] > 0.0 && mylast < 0) mylast = v0 + tid * 4 + e;
    }
    if (mine != 0x7fffffff) atomicMin(&sh.tok, mine);
    if (mylast >= 0) atomicMax(&sh.last, mylast);
    __syncthreads();
    const int token = sh.tok != 0x7fffffff ? sh.tok : sh.last;
    if (!PRECISE && use_resid && Q > 0.0) {
        // with q~ present the thresholds depend on the normaliser: error <= GUARD_Z * Q
        const double E2 = 2.0 * GUARD_Z * Q;
        if (sh.tok == 0x7fffffff) {
            if (tid == 0) sh.flag = 1;
        } else if (mine == sh.tok) {
            const int e = mine - (v0 + tid * 4);
            const double hi = base + cum[e] - thr2;
            const double lo = thr2 - (base + cum[e] - r[e]);
            if (hi < E2 || lo < E2) sh.flag = 1;
        }
    }
    __syncthreads();
    return token;
}

// One sequence (fast pass: sequence `slot`; double-precision pass: entry `slot` of the queue), by the
// 256 threads of a CTA.  cm: [nch] doubles of shared memory (chunk masses of the sampled row).
// SHARDED: vocabulary-parallel verification (a.entry_logits and a.pick are set).
template <typename T, bool PRECISE, bool SHARDED>
__device__ __forceinline__ void verify_finish_slot(const VerifyArgs& a, int slot, FinishShared& sh, double* cm) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = a.G, G1 = a.G + 1;
    {
        // a queue entry is the sequence, with QUEUE_DRAW_ONLY set when only the draw was too close to
        // call: then the accept decisions of the fast pass stand and only the sampled row is redone;
        // with QUEUE_MASS_ONLY every decision stands and only small residual masses are recomputed
        const int qe = PRECISE ? a.queue[slot] : slot;
        const int b = PRECISE ? (qe & QUEUE_SEQ_MASK) : slot;
        const bool draw_only = PRECISE && (qe & QUEUE_DRAW_ONLY) != 0;
        const bool mass_only = PRECISE && (qe & QUEUE_MASS_ONLY) != 0;
        const int alen_fast = draw_only ? a.accept_len[b] : 0;
        const unsigned long long need = PRECISE ? a.need_rows[b] : 0ull;   // rows with exact chunk sums
        if (!a.sample_only && a.state_in && a.state_in[b] == 0) {
            // decided by an earlier call: nothing of this sequence is read or written
            if (tid == 0 && a.state_out) a.state_out[b] = 0;
            return;
        }
        const float Tb = a.temperature[b];
        const float c32 = temp_scale(Tb);
        const T* seq = reinterpret_cast<const T*>(a.logits) + (long long)b * G1 * a.row_stride;
        unsigned st_bits = 0;
        if (!temp_ok(Tb)) st_bits |= ST_TEMPERATURE;
        // (requested now, looked at when the outputs are written)
        const unsigned status_word = *(volatile unsigned*)a.status;
        // the two uniforms of the draw, requested long before the chunk masses are ready
        const float u_chunk = a.u_resample ? a.u_resample[2 * b] : 0.f;
        const float u_entry = a.u_resample ? a.u_resample[2 * b + 1] : 0.f;
        // rows lo .. row_hi-1 are read, positions lo .. hi-1 are tested; g is the bonus row
        const int lo = a.sample_only ? 0 : a.r0;
        const int g = (!a.sample_only && a.gamma) ? a.gamma[b] : G;
        if (g < 0 || g > G || g < lo) st_bits |= ST_RANGE;
        const int hi = a.sample_only ? G : min(g, a.r1);
        const int row_hi = a.sample_only ? G1 : min(g + 1, a.r1);
        __syncthreads();
        if (tid == 0) {
            sh.bad = 0;
            sh.flag = 0;
        }
        __syncthreads();

        // ---- 1. normaliser of every row that is needed ------------------------------------
        int jpos = -1;
        if (a.sample_only) {
            jpos = a.pos[b];
            if (jpos < 0 || jpos > G) st_bits |= ST_RANGE;
        }
        if (!st_bits) {
            const int i_lo = a.sample_only ? jpos : lo, i_hi = a.sample_only ? jpos + 1 : row_hi;
            for (int i = i_lo + warp; i < i_hi; i += WARPS) {
                if (draw_only && i != alen_fast) continue;
                if (mass_only && !row_needed(need, i)) continue;
                double Z, Zraw;
                float mx;
                bool bad;
                row_stats<T>(a, b * G1 + i, c32, lane, PRECISE && row_needed(need, i), Z, Zraw, mx, bad);
                if (lane == 0) {
                    sh.Z[i] = Z;
                    sh.Zraw[i] = Zraw;
                    sh.mx[i] = mx;
                    if (!PRECISE) a.row_max[b * G1 + i] = mx;
                    if (bad) atomicOr(&sh.bad, (int)ST_LOGIT);
                }
            }
        }
        __syncthreads();

        // ---- 2. per draft position: p(x), q~(x), accept test, residual mass ----------------
        if (!st_bits && !sh.bad && !a.sample_only && !draw_only) {
            for (int i = lo + warp; i < hi; i += WARPS) {
                if (mass_only && !row_needed(need, i)) continue;
                const int ri = b * G + i;
                const int* idx = a.q_idx + (long long)ri * a.k_max;
                const float* prob = a.q_prob + (long long)ri * a.k_max;
                const T* row = seq + (long long)i * a.row_stride;
                // the first batch of stored entries is requested before the row's count is known
                // (every slot below k_max exists; slots at or beyond the count are dropped below)
                int vv[8];
                float qq[8], ll[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int k = u * 32 + lane;
                    vv[u] = k < a.k_max ? idx[k] : -2;
                    qq[u] = k < a.k_max ? prob[k] : 0.f;
                }
                const int x = a.draft_tok[ri];
                const int n = a.q_count[ri];
                const float ux = a.u_accept[ri];
                bool range_bad = (x < 0 || x >= a.V || n < 0 || n > a.k_max);
                Weight<PRECISE> wt;
                wt.init(Tb, sh.mx[i]);
                const double Z = sh.Z[i];
                const double invZ = 1.0 / Z;     // the sums below take p = w * (1/Z): 2^-53 relative per term
                double smin = 0.0;
                float qx = 0.f, qx_mine = 0.f;
                int kx = 0x7fffffff;
                // p(x) on every lane (the same instructions as on one lane, and no divergent tail)
                const float* ent = SHARDED ? a.entry_logits + (long long)ri * (a.k_max + 1) : nullptr;
                const float lx = range_bad ? -CUDART_INF_F : (SHARDED ? ent[a.k_max] : load_logit(row, x));
                if (!range_bad) {
                    for (int k0 = 0; k0 < n; k0 += 256) {
                        if (k0 > 0) {
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                const int k = k0 + u * 32 + lane;
                                vv[u] = k < n ? idx[k] : -2;
                                qq[u] = k < n ? prob[k] : 0.f;
                            }
                        }
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            if (k0 + u * 32 + lane >= n) vv[u] = -2;
                            const bool ok = vv[u] >= 0 && vv[u] < a.V;
                            if (vv[u] != -2 && !ok) range_bad = true;
                            ll[u] = ok ? (SHARDED ? ent[k0 + u * 32 + lane] : load_logit(row, vv[u])) : -CUDART_INF_F;
                        }
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const int k = k0 + u * 32 + lane;
                            if (vv[u] >= 0 && vv[u] < a.V) {
                                const double pk = wt(ll[u]) * invZ;
                                smin += fmin(pk, (double)qq[u]);
                                if (vv[u] == x && k < kx) {
                                    kx = k;
                                    qx_mine = qq[u];
                                }
                            }
                        }
                    }
                }
                const double px = wt(lx) / Z;
                range_bad = __any_sync(0xffffffffu, range_bad);
                smin = warp_sum(smin);
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) kx = min(kx, __shfl_xor_sync(0xffffffffu, kx, d));
                // the stored probability of the first entry that names the draft token sits in lane kx % 32
                qx = __shfl_sync(0xffffffffu, qx_mine, kx & 31);
                if (kx == 0x7fffffff) qx = 0.f;
                if (lane == 0) {
                    if (range_bad) {
                        atomicOr(&sh.bad, (int)ST_RANGE);
                    } else {
                        const double u = (double)ux;
                        int acc = 1, amb = 0, bord = 0;
                        if (qx > 0.f) {
                            const double ratio = px / (double)qx;
                            acc = u < fmin(1.0, ratio);
                            const double dist = fabs(ratio - u);
                            if (PRECISE)
                                bord = dist <= BORDER_REL * u;
                            else
                                amb = dist <= (BORDER_REL + GUARD_Z) * fmax(u, ratio);
                        }
                        sh.acc[i] = acc;
                        sh.amb[i] = amb;
                        sh.bord[i] = bord;
                        double R = 1.0 - smin;
                        if (R < 0.0) R = 0.0;
                        // 1 - sum min(p, q~) inherits the absolute error of the fp32-accumulated
                        // normaliser: a small residual mass is reported from the exact sums instead
                        sh.small[i] = !PRECISE && R < RESID_EXACT_BELOW;
                        a.p_draft[ri] = (float)px;
                        a.resid_mass[ri] = (float)R;
                    }
                }
            }
        }
        __syncthreads();
        st_bits |= (unsigned)sh.bad;
        if (mass_only) return;          // (bad data was reported by the fast pass already)

        // ---- 3. first-rejection scan -----------------------------------------------------
        // A rejection inside the range decides the sequence; so does accepting every position
        // when the bonus row g is in the range.  Otherwise it waits for the next rows.
        int alen = lo, nborder = 0;
        bool flagged = false, rejected = false, decided = true;
        if (draw_only) {
            // (no accept test was ambiguous, so none is borderline either)
            alen = alen_fast;
            rejected = alen < hi;
        } else if (!st_bits && !a.sample_only) {
            while (alen < hi && sh.acc[alen]) ++alen;
            rejected = alen < hi;
            decided = rejected || g < a.r1;
            const int last = rejected ? alen : hi - 1;
            for (int i = lo; i <= last; ++i) {
                flagged |= sh.amb[i] != 0;
                nborder += sh.bord[i];
            }
            if (!PRECISE)
                for (int i = lo; i < hi; ++i) flagged |= sh.small[i] != 0;
        }

        // ---- 4. residual / bonus sample --------------------------------------------------
        int token = -1;
        int pick_row = 0, pick_chunk = -1;      // vocabulary-parallel: what the picked chunk's owner needs
        bool pick_resid = false;
        double Rtot = -1.0;
        const bool want_token = SHARDED || a.token != nullptr;
        if (!st_bits && want_token && decided) {
            const int j = a.sample_only ? jpos : alen;
            const int rj = b * G + j;
            int n = 0;
            if (a.sample_only ? j < G : rejected) {
                n = a.q_count[rj];
                if (n < 0 || n > a.k_max) {
                    n = 0;
                    st_bits |= ST_RANGE;
                }
            }
            const int* idx = a.q_idx + (long long)rj * a.k_max;
            const float* prob = a.q_prob + (long long)rj * a.k_max;
            const T* row = seq + (long long)j * a.row_stride;
            Weight<PRECISE> wt;
            wt.init(Tb, sh.mx[j]);
            const double Z = sh.Z[j];
            const double invZ = 1.0 / Z;
            bool use_resid = n > 0;
            for (int pass = 0; pass < 2 && !st_bits; ++pass) {
                // chunk masses (in units where the row sums to one)
                if (PRECISE && row_needed(need, j)) {
                    for (int c = tid; c < a.nch; c += THREADS) cm[c] = a.dsum[record_index(a, b * G1 + j, c)] * invZ;
                } else {
                    const double off = (double)__fmul_rn(sh.mx[j], c32);
                    const double Zraw = sh.Zraw[j];
                    for (int c = tid; c < a.nch; c += THREADS) {
                        float2 v = a.stats[record_index(a, b * G1 + j, c)];
                        cm[c] = v.x > -CUDART_INF_F ? (double)v.y * exp2((double)__fmul_rn(v.x, c32) - off) / Zraw : 0.0;
                    }
                }
                __syncthreads();
                if (use_resid) {
                    bool rb = false;
                    {
                        // n <= 1024: at most four entries per thread, loads first
                        int vv[4];
                        float qq[4], ll[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int k = tid + u * THREADS;
                            vv[u] = k < n ? idx[k] : -2;
                            qq[u] = k < n ? prob[k] : 0.f;
                        }
                        const float* ent = SHARDED ? a.entry_logits + (long long)rj * (a.k_max + 1) : nullptr;
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const bool ok = vv[u] >= 0 && vv[u] < a.V;
                            if (vv[u] != -2 && !ok) rb = true;
                            ll[u] = ok ? (SHARDED ? ent[tid + u * THREADS] : load_logit(row, vv[u])) : -CUDART_INF_F;
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            if (vv[u] >= 0 && vv[u] < a.V)
                                atomicAdd(&cm[vv[u] / CHUNK], -fmin(wt(ll[u]) * invZ, (double)qq[u]));
                    }
                    if (rb) atomicOr(&sh.bad, (int)ST_RANGE);
                }
                __syncthreads();
                // level 1 by warp 0: lanes own contiguous blocks of chunks
                if (warp == 0) {
                    const int per = (a.nch + 31) / 32;
                    const int c0 = lane * per, c1 = min(a.nch, c0 + per);
                    double s = 0.0;
                    for (int c = c0; c < c1; ++c) {
                        double m = cm[c];
                        if (m < 0.0) {
                            m = 0.0;
                            cm[c] = 0.0;
                        }
                        s += m;
                    }
                    double incl = s;
#pragma unroll
                    for (int d = 1; d < 32; d <<= 1) {
                        double y = __shfl_up_sync(0xffffffffu, incl, d);
                        if (lane >= d) incl += y;
                    }
                    const double R = __shfl_sync(0xffffffffu, incl, 31);
                    const double thr = (double)u_chunk * R;
                    double run = incl - s;
                    int first = 0x7fffffff, lastpos = -1;
                    double mind = 1e300;
                    for (int c = c0; c < c1; ++c) {
                        const double m = cm[c];
                        run += m;
                        if (m > 0.0) lastpos = c;
                        if (run > thr && first == 0x7fffffff) first = c;
                        mind = fmin(mind, fabs(run - thr));
                    }
#pragma unroll
                    for (int d = 16; d > 0; d >>= 1) {
                        first = min(first, __shfl_xor_sync(0xffffffffu, first, d));
                        lastpos = max(lastpos, __shfl_xor_sync(0xffffffffu, lastpos, d));
                        mind = fmin(mind, __shfl_xor_sync(0xffffffffu, mind, d));
                    }
                    if (lane == 0) {
                        sh.cstar = first != 0x7fffffff ? first : lastpos;
                        sh.Rtot = R;
                        // every prefix and the total carry an absolute error <= GUARD_Z
                        if (!PRECISE && mind <= GUARD_Z) sh.flag = 1;
                    }
                }
                __syncthreads();
                Rtot = sh.Rtot;
                if (!use_resid) break;
                // the residual may vanish (q~ >= p everywhere): then the draw is from p itself
                const double tiny = PRECISE ? RESID_ZERO_BELOW : 4.0 * GUARD_Z;
                // (a reported mass this small would show the normaliser's error: exact sums instead)
                if (!PRECISE && a.mass && Rtot < RESID_EXACT_BELOW && tid == 0) sh.flag = 1;
                if (Rtot > tiny) break;
                if (!PRECISE) {
                    if (tid == 0) sh.flag = 1;   // too close to zero to call in fp32
                    break;
                }
                use_resid = false;  // precise: residual is zero, fall back to p
                __syncthreads();
            }
            st_bits |= (unsigned)sh.bad;
            const int cs = st_bits ? -1 : sh.cstar;
            pick_row = j;
            pick_chunk = cs;
            pick_resid = use_resid;
            if (!st_bits && cs >= 0 && !SHARDED) {
                token = level2_draw<T, PRECISE>(a, row, 0, cs, idx, prob, n, use_resid, wt, invZ,
                                                u_entry, sh);
            }
            flagged |= sh.flag != 0;
        }

        // ---- 5. outputs --------------------------------------------------------------------
        // a wait of the streaming pass ran out (now or in a call since the status word was last
        // cleared): its statistics are not complete, nothing of this call is valid
        if (status_word & ST_INTERNAL) st_bits |= ST_INTERNAL;
        if (tid == 0) {
            if (st_bits) {
                atomicOr(a.status, st_bits);
                if (!a.sample_only) {
                    a.accept_len[b] = -1;
                    for (int i = lo; i < hi && i < G; ++i) {
                        a.p_draft[b * G + i] = -1.f;
                        a.resid_mass[b * G + i] = -1.f;
                    }
                    if (a.state_out) a.state_out[b] = 0;
                }
                if (a.token) a.token[b] = -1;
                if (SHARDED) {
                    a.pick[4 * b + 0] = 0;
                    a.pick[4 * b + 1] = -1;
                    a.pick[4 * b + 2] = 0;
                }
                if (a.mass) a.mass[b] = -1.f;
            } else {
                if (!a.sample_only) {
                    a.accept_len[b] = decided ? alen : -2;
                    if (a.state_out) a.state_out[b] = decided ? 0 : 1;
                }
                if (a.token) a.token[b] = decided ? token : -2;
                if (a.mass) a.mass[b] = (float)Rtot;
                if (PRECISE) {
                    if (nborder && a.borderline) atomicAdd(a.borderline, nborder);
                    if (SHARDED) {
                        a.pick[4 * b + 0] = pick_row;
                        a.pick[4 * b + 1] = (decided && want_token) ? pick_chunk : -1;
                        a.pick[4 * b + 2] = pick_resid ? PICK_RESIDUAL : 0;
                    }
                } else if (flagged || SHARDED) {
                    // Which rows need exact sums: an ambiguous accept test can move the first
                    // rejection anywhere from its position on, so every row from there; an ambiguous
                    // draw needs the sampled row only; a small residual mass its own row.
                    unsigned long long nd = 0ull;
                    int nrows = 0;
                    bool draw_only_flag = false, mass_only_flag = false;
                    if (a.sample_only) {
                        nd = ~0ull;
                        nrows = 1;
                        a.rowq[atomicAdd(a.rowq_count, 1)] = b * G1 + jpos;
                    } else {
                        int first_amb = -1;
                        const int last = rejected ? alen : hi - 1;
                        for (int i = lo; i <= last && first_amb < 0; ++i)
                            if (sh.amb[i]) first_amb = i;
                        bool any_small = false;
                        for (int i = lo; i < hi; ++i) any_small |= sh.small[i] != 0;
                        draw_only_flag = first_amb < 0 && !any_small;
                        mass_only_flag = first_amb < 0 && any_small && !sh.flag;
                        for (int i = lo; i < row_hi; ++i) {
                            // (vocabulary-parallel: whether the draw inside the chunk is too close to call is
                            // only known to the chunk's owner later, so the sampled row is always listed)
                            const bool nr = i >= 64 || (first_amb >= 0 && i >= first_amb) || (i < hi && sh.small[i]) ||
                                            ((sh.flag || SHARDED) && want_token && decided && i == alen);
                            if (nr) {
                                if (i < 64) nd |= 1ull << i;
                                ++nrows;
                                if (!SHARDED) a.rowq[atomicAdd(a.rowq_count, 1)] = b * G1 + i;
                            }
                        }
                    }
                    a.need_rows[b] = nd;
                    if (SHARDED) {
                        // the queue is built once the owners' flags have been exchanged
                        a.pick[4 * b + 0] = pick_row;
                        a.pick[4 * b + 1] = (decided && want_token) ? pick_chunk : -1;
                        a.pick[4 * b + 2] = (pick_resid ? PICK_RESIDUAL : 0) | (flagged ? PICK_FLAGGED : 0) |
                                            (draw_only_flag ? PICK_DRAW_ONLY : 0) | (mass_only_flag ? PICK_MASS_ONLY : 0);
                        a.pick[4 * b + 3] = nrows;
                    } else {
                        const int q = atomicAdd(a.queue_count, 1);
                        a.queue[q] = b | (draw_only_flag ? QUEUE_DRAW_ONLY : 0) | (mass_only_flag ? QUEUE_MASS_ONLY : 0);
                        atomicAdd(a.slow_rows, (unsigned long long)nrows);
                    }
                }
            }
        }
    }
}

template <typename T, bool PRECISE, bool SHARDED = false>
__global__ void __launch_bounds__(THREADS, 2) verify_finish_kernel(VerifyArgs a) {
    extern __shared__ double cm[];  // [nch] chunk masses of the sampled row
    __shared__ FinishShared sh;
    grid_dependency_sync();
    const int nloop = PRECISE ? *a.queue_count : a.B;
    for (int slot = blockIdx.x; slot < nloop; slot += gridDim.x) verify_finish_slot<T, PRECISE, SHARDED>(a, slot, sh, cm);
}

}  // namespace picospec
