// Draft-side kernels: one streaming pass per row that keeps the top-k candidates under the
// order (logit descending, index ascending) in shared memory, then top-p cut, renormalisation,
// emission and the optional draft-token draw.
#pragma once
#include "common.cuh"
#include "precise_kernels.cuh"

namespace picospec {

typedef unsigned long long u64;

struct CsRowMeta;   // per-row record the staged filter kernel leaves for its finish kernel

constexpr int ITER_ELEMS = WARPS * CHUNK;            // entries one CTA iteration can push at most
constexpr int CAND_CAP = ITER_ELEMS + 2 * MAX_K;     // candidate buffer (keys)
constexpr int COMPRESS_SMEM = CAND_CAP * 8 + MAX_K * 8;   // candidate keys + staging / sorted keys

struct CompressArgs {
    const void* logits;        // draft logits [B, G, V]
    long long row_stride;
    int B, G, V, nch, k_max, top_k;
    float top_p;
    const float* temperature;
    int* q_idx;
    float* q_prob;
    int* q_count;
    const float* u_draft;      // or null
    int* draft_tok;            // or null
    // workspace
    float* row_max;            // [B*G]
    double* dsum;              // [B*G, nch]
    int* queue;
    int* queue_count;          // zero on entry (cleared by the previous call)
    int* queue_count_next;     // cleared by this call for the next one
    int* tickets;              // per queue slot: chunk sums completed in the double-precision pass
    unsigned* status;
    unsigned long long* slow_rows;
    // rows the staged kernel hands to the direct kernel (candidate buffer overflow)
    int* redo_rows;            // [B*G]
    int* redo_count;           // zero on entry of the staged kernel
    int* redo_count_next;      // cleared for the next call
    int use_redo_list;         // direct kernel: 1 = process redo_rows[0 .. *redo_count) only
    unsigned long long* redo_total;   // cumulative number of rows handed over (reported by picospec_counters)
    // Top-K of selected rows (picospec_target_topk): output row r reads logits row
    // r * seq_rows + row_pos[r]; probabilities are emitted as they are (divided by the row's
    // normaliser, not by the mass of the kept entries)
    const int* row_pos;        // or null: output row r reads logits row r
    int seq_rows;
    int raw_probs;
    // staged path: survivors of the filter kernel, [B*G, cs_survivor_cap(k_max)] keys + one record per row
    unsigned long long* surv_keys;
    CsRowMeta* surv_meta;
};

// logits row behind output row `row`, or -1 if its position is out of range
__device__ __forceinline__ long long source_row(const CompressArgs& a, int row) {
    if (!a.row_pos) return row;
    const int j = a.row_pos[row];
    return (j < 0 || j >= a.seq_rows) ? -1 : (long long)row * a.seq_rows + j;
}

// Monotone map float -> uint32 (larger float, larger key); -0 is folded onto +0 so that the two
// zeros tie as they do under a floating-point comparison.
__device__ __forceinline__ uint32_t orderable(float f) {
    uint32_t b = __float_as_uint(f);
    if (b == 0x80000000u) b = 0u;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float from_orderable(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
// larger key = earlier in the order (logit descending, index ascending)
__device__ __forceinline__ u64 make_key(float l, int v) {
    return ((u64)orderable(l) << 32) | (u64)(0xFFFFFFFFu - (uint32_t)v);
}
__device__ __forceinline__ int key_index(u64 k) { return (int)(0xFFFFFFFFu - (uint32_t)k); }
__device__ __forceinline__ float key_logit(u64 k) { return from_orderable((uint32_t)(k >> 32)); }

struct CompressShared {
    int hist[256];
    int count;
    float thr;
    int nan;
    u64 prefix;
    int krem;
    int n, first, last, flag;
    double Wn;
    double warp_tot[WARPS];
    float wM[WARPS];
    double wS[WARPS];
};

// k-th largest of keys[0..count) (1 <= k <= count), CTA-wide MSD radix select, 8 bits per pass.
// LOGIT16: bf16 data, the two passes over the low 16 bits of the logit part are skipped.
// The top byte of the index part is always 0xFF (V <= 2^22), one more pass is skipped.
template <bool LOGIT16>
__device__ u64 radix_select_kth(const u64* keys, int count, int k, CompressShared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        sh.prefix = 0ull;
        sh.krem = k;
    }
    u64 mask = 0ull;
    for (int shift = 56; shift >= 0; shift -= 8) {
        // passes whose digit is known in advance: for bf16 data the low 16 bits of the logit part
        // are 0x0000 (non-negative logits, top key bit set) or 0xFFFF (negative logits, whose
        // orderable form is the complement); the top byte of the index part is 0xFF
        const bool logit_low = LOGIT16 && (shift == 40 || shift == 32);
        if (logit_low || shift == 24) {
            workers_sync();
            if (tid == 0) {
                const u64 digit = (shift == 24 || !(sh.prefix >> 63)) ? 0xFFull : 0x00ull;
                sh.prefix |= digit << shift;
            }
            mask |= 0xFFull << shift;
            continue;
        }
        sh.hist[tid] = 0;
        workers_sync();
        const u64 prefix = sh.prefix;
        for (int i = tid; i < count; i += THREADS) {
            const u64 key = keys[i];
            if ((key & mask) == prefix) atomicAdd(&sh.hist[(int)((key >> shift) & 0xFF)], 1);
        }
        workers_sync();
        if (warp == 0) {
            int loc[8], s = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                loc[j] = sh.hist[255 - 8 * lane - j];
                s += loc[j];
            }
            int incl = s;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                int y = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += y;
            }
            const int excl = incl - s, krem = sh.krem;
            if (excl < krem && krem <= incl) {
                int run = excl;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (run + loc[j] >= krem) {
                        sh.krem = krem - run;
                        sh.prefix = prefix | ((u64)(255 - 8 * lane - j) << shift);
                        break;
                    }
                    run += loc[j];
                }
            }
        }
        mask |= 0xFFull << shift;
        workers_sync();
    }
    workers_sync();
    return sh.prefix;
}

// Keep the k largest keys of cand[0..count): afterwards cand[0..k) holds them (unordered).
template <bool LOGIT16>
__device__ u64 keep_top_k(u64* cand, u64* keep, int count, int k, CompressShared& sh) {
    const u64 kth = radix_select_kth<LOGIT16>(cand, count, k, sh);
    workers_sync();
    if (threadIdx.x == 0) sh.count = 0;
    workers_sync();
    for (int i = threadIdx.x; i < count; i += THREADS) {
        const u64 key = cand[i];
        if (key >= kth) keep[atomicAdd(&sh.count, 1)] = key;   // keys are distinct: exactly k pass
    }
    workers_sync();
    for (int i = threadIdx.x; i < k; i += THREADS) cand[i] = keep[i];
    workers_sync();
    return kth;
}

// Descending bitonic sort of keys[0..n2), n2 a power of two, by the 256 workers.  Thread t takes the
// compare-exchange pairs t, t + 256, ...; with a stride of at most 32 the 32 pairs of a warp
// stay inside one aligned block of 64 keys that no other warp touches in that stage, so those stages
// only need a warp-level sync; a CTA barrier separates them from the stages with longer strides.
__device__ void bitonic_sort_desc(u64* keys, int n2) {
    bool cross = true;      // the previous stage (or the caller's writes) crossed warp blocks
    for (int size = 2; size <= n2; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const bool local = stride <= 32;
            if (!local || cross) workers_sync();
            else __syncwarp();
            cross = !local;
            for (int i = threadIdx.x; i < (n2 >> 1); i += THREADS) {
                const int pos = 2 * i - (i & (stride - 1));
                const int j = pos + stride;
                const bool desc = (pos & size) == 0;
                const u64 x = keys[pos], y = keys[j];
                if ((x < y) == desc) {
                    keys[pos] = y;
                    keys[j] = x;
                }
            }
        }
    }
    workers_sync();
}

__device__ __forceinline__ void emit_invalid_row(const CompressArgs& a, int row) {
    for (int j = threadIdx.x; j < a.k_max; j += THREADS) {
        a.q_idx[(long long)row * a.k_max + j] = -1;
        a.q_prob[(long long)row * a.k_max + j] = 0.f;
    }
    if (threadIdx.x == 0) {
        a.q_count[row] = -1;
        if (a.draft_tok) a.draft_tok[row] = -1;
    }
}

// Top-p cut, renormalisation, emission and draft draw for one row whose k_eff best candidates
// sit sorted in keys[0..k_eff).  Z is the row normaliser on the scale of Weight<PRECISE>
// (ignored when top_p >= 1).  Returns (to thread 0, via sh.flag) whether the cut was too close
// to call in the fast path.
template <bool PRECISE, int E>
__device__ void finish_row_ranks(const CompressArgs& a, int row, const u64* keys, int k_eff, float Tb, double Z,
                           CompressShared& sh) {
    const int tid = threadIdx.x;
    const float mx = key_logit(keys[0]);
    Weight<PRECISE> wt;
    wt.init(Tb, mx);
    if (tid == 0) {
        sh.first = 0x7fffffff;
        sh.last = -1;
        sh.flag = 0;
        sh.n = k_eff;
    }
    // E consecutive ranks per thread
    double w[E], cum[E], loc = 0.0;
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const int j = tid * E + e;
        w[e] = j < k_eff ? wt(key_logit(keys[j])) : 0.0;
        loc += w[e];
        cum[e] = loc;
    }
    double Wtot;
    const double base = block_scan_incl(loc, sh.warp_tot, Wtot) - loc;   // syncs: sh.first is set
    if (a.top_p < 1.0f) {
        const double thrZ = (double)a.top_p * Z;
        int mine = 0x7fffffff;
#pragma unroll
        for (int e = E - 1; e >= 0; --e)
            if (tid * E + e < k_eff && base + cum[e] >= thrZ) mine = tid * E + e;
        if (mine != 0x7fffffff) atomicMin(&sh.first, mine);
        workers_sync();
        const int jn = sh.first;   // rank of the entry that reaches top_p, if any
        if (jn != 0x7fffffff && jn == mine) {
            sh.n = jn + 1;
            if (!PRECISE) {
                const int e = jn - tid * E;
                const double E = GUARD_Z * thrZ;
                const double hi = base + cum[e] - thrZ;
                const double lo = thrZ - (base + cum[e] - w[e]);
                // reaching top_p one entry earlier or later changes n unless the cap hides it
                if ((hi < E && jn + 1 < k_eff) || (lo <= E && jn > 0)) sh.flag = 1;
            }
        }
        if (!PRECISE && jn == 0x7fffffff && tid == 0) {
            // never reached: n = k_eff either way, nothing to decide
        }
        workers_sync();
    }
    const int n = sh.n;
#pragma unroll
    for (int e = 0; e < E; ++e)
        if (tid * E + e == n - 1) sh.Wn = base + cum[e];
    workers_sync();
    const double Wn = sh.Wn;
    // stored probabilities, and their running sum for the draft draw
    float pf[E];
    double ploc = 0.0, pcum[E];
    const double inv = 1.0 / (a.raw_probs ? Z : Wn);   // one division per row; 2^-53 relative per entry
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const int j = tid * E + e;
        pf[e] = j < n ? (float)(w[e] * inv) : 0.f;
        ploc += (double)pf[e];
        pcum[e] = ploc;
    }
    const bool flagged = !PRECISE && sh.flag;
    long long o = (long long)row * a.k_max;
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const int j = tid * E + e;
        if (j < a.k_max) {
            // a flagged row keeps all k_eff sorted candidates so that the double-precision pass
            // can redo the cut without a second selection
            const bool keep_idx = j < n || (flagged && j < k_eff);
            a.q_idx[o + j] = keep_idx ? key_index(keys[j]) : -1;
            a.q_prob[o + j] = pf[e];
        }
    }
    for (int j = THREADS * E + tid; j < a.k_max; j += THREADS) {   // slots beyond the ranks the threads hold
        a.q_idx[o + j] = -1;
        a.q_prob[o + j] = 0.f;
    }
    if (a.draft_tok) {
        if (tid == 0) {
            sh.first = 0x7fffffff;
            sh.last = -1;
        }
        double Ptot;
        const double pbase = block_scan_incl(ploc, sh.warp_tot, Ptot) - ploc;
        const double thr = (double)a.u_draft[row] * Ptot;
        int mine = 0x7fffffff, mylast = -1;
#pragma unroll
        for (int e = E - 1; e >= 0; --e) {
            if (tid * E + e < n && pbase + pcum[e] > thr) mine = tid * E + e;
            if (pf[e] > 0.f && mylast < 0) mylast = tid * E + e;
        }
        if (mine != 0x7fffffff) atomicMin(&sh.first, mine);
        if (mylast >= 0) atomicMax(&sh.last, mylast);
        workers_sync();
        if (tid == 0) {
            const int j = sh.first != 0x7fffffff ? sh.first : sh.last;
            a.draft_tok[row] = j >= 0 ? key_index(keys[j]) : -1;
        }
    }
    if (tid == 0) {
        a.q_count[row] = n;
        if (flagged) {
            a.row_max[row] = mx;
            const int q = atomicAdd(a.queue_count, 1);
            a.queue[q] = row;
            a.tickets[q] = 0;
            atomicAdd(a.slow_rows, 1ull);
        }
    }
    workers_sync();
}

// (the ranks are spread over as many threads as there are: one per thread up to 256 candidates,
// which shortens the serial part -- the exponentials and the running sums -- fourfold)
template <bool PRECISE>
__device__ __forceinline__ void finish_row(const CompressArgs& a, int row, const u64* keys, int k_eff, float Tb, double Z,
                                           CompressShared& sh) {
    if (k_eff <= THREADS) finish_row_ranks<PRECISE, 1>(a, row, keys, k_eff, Tb, Z, sh);
    else if (k_eff <= 2 * THREADS) finish_row_ranks<PRECISE, 2>(a, row, keys, k_eff, Tb, Z, sh);
    else finish_row_ranks<PRECISE, 4>(a, row, keys, k_eff, Tb, Z, sh);
}

template <typename T, bool ALIGNED, bool STATS>
__global__ void __launch_bounds__(THREADS, 2) compress_kernel(CompressArgs a) {
    grid_dependency_sync();
    extern __shared__ u64 smem64[];
    u64* cand = smem64;
    u64* keep = cand + CAND_CAP;
    __shared__ CompressShared sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr bool LOGIT16 = sizeof(T) == 2;
    const int rows = a.B * a.G;
    const int iters = (a.nch + WARPS - 1) / WARPS;
    int k_eff = a.top_k > 0 ? a.top_k : a.k_max;
    if (k_eff > a.k_max) k_eff = a.k_max;
    if (k_eff > a.V) k_eff = a.V;

    // a call that goes through this kernel alone clears both of the next call's counters, as the
    // staged filter kernel does (the redo-list launch of a staged call must not: the filter did)
    if (blockIdx.x == 0 && tid == 0 && !a.use_redo_list) {
        *a.queue_count_next = 0;
        *a.redo_count_next = 0;
    }
    const int nwork = a.use_redo_list ? *a.redo_count : rows;

    for (int wi = blockIdx.x; wi < nwork; wi += gridDim.x) {
        const int row = a.use_redo_list ? a.redo_rows[wi] : wi;
        const int b = row / a.G;
        const float Tb = a.temperature[b];
        workers_sync();
        if (!temp_ok(Tb)) {
            emit_invalid_row(a, row);
            if (tid == 0) atomicOr(a.status, ST_TEMPERATURE);
            continue;
        }
        const float c32 = temp_scale(Tb);
        const long long srow = source_row(a, row);
        if (srow < 0) {
            emit_invalid_row(a, row);
            if (tid == 0) atomicOr(a.status, ST_RANGE);
            continue;
        }
        const T* rowp = reinterpret_cast<const T*>(a.logits) + srow * a.row_stride;
        if (tid == 0) {
            sh.count = 0;
            sh.thr = -CUDART_INF_F;
            sh.nan = 0;
        }
        workers_sync();

        // running softmax statistics of this warp: fp32 lane sums relative to the warp's running
        // maximum; when the maximum rises the sums are folded into a double and rescaled exactly
        float runM = -CUDART_INF_F, runOff = 0.f, acc = 0.f;
        double folded = 0.0;

        ChunkRegs<T> bufA, bufB;
        if (warp < a.nch) bufA.template load<ALIGNED>(rowp, warp * CHUNK, a.V, lane);
        auto body = [&](ChunkRegs<T>& cur, ChunkRegs<T>& nxt, int it) {
            const int c = it * WARPS + warp;
            const int cn = c + WARPS;
            if (it + 1 < iters && cn < a.nch) nxt.template load<ALIGNED>(rowp, cn * CHUNK, a.V, lane);
            const float thr = sh.thr;
            if (c < a.nch) {
                const int v0 = c * CHUNK;
                const float lm = cur.lane_max();
                if (lm != lm) sh.nan = 1;
                if (STATS) {
                    const float cmx = warp_max(lm);
                    if (cmx > runM) {
                        const float newOff = __fmul_rn(cmx, c32);
                        const double s = (double)warp_sum(acc);
                        folded = runM > -CUDART_INF_F ? (folded + s) * exp2((double)runOff - (double)newOff) : 0.0;
                        acc = 0.f;
                        runM = cmx;
                        runOff = newOff;
                    }
                    if (runM > -CUDART_INF_F && runM < CUDART_INF_F) acc += lane_exp_sum(cur, c32, runOff);
                }
                if (lm >= thr) {
#pragma unroll
                    for (int j = 0; j < ChunkRegs<T>::NVEC; ++j) {
                        if (cur.vec_max(j) >= thr) {
                            constexpr int VEC = ChunkRegs<T>::VEC;
#pragma unroll
                            for (int e = 0; e < VEC; ++e) {
                                const float l = cur.value(j * VEC + e);
                                const int v = v0 + ChunkRegs<T>::offset(j * VEC + e, lane);
                                if (l >= thr && v < a.V) cand[atomicAdd(&sh.count, 1)] = make_key(l, v);
                            }
                        }
                    }
                }
            }
            workers_sync();
            if (sh.count > CAND_CAP - ITER_ELEMS) {
                const int count = sh.count;
                workers_sync();
                keep_top_k<LOGIT16>(cand, keep, count, k_eff, sh);
                // sh.count == k_eff now; the k-th key's logit is the new admission threshold
                float mn = CUDART_INF_F;
                for (int i = tid; i < k_eff; i += THREADS) mn = fminf(mn, key_logit(cand[i]));
                mn = -warp_max(-mn);
                if (lane == 0) sh.wM[warp] = mn;
                workers_sync();
                if (tid == 0) {
                    float m = sh.wM[0];
                    for (int w = 1; w < WARPS; ++w) m = fminf(m, sh.wM[w]);
                    sh.thr = m;
                }
                workers_sync();
            }
        };
        for (int it = 0; it < iters; it += 2) {
            body(bufA, bufB, it);
            if (it + 1 < iters) body(bufB, bufA, it + 1);
        }

        // ---- row statistics -----------------------------------------------------------------
        double Z = 0.0;
        if (STATS) {
            const double s = (double)warp_sum(acc);
            if (lane == 0) {
                sh.wM[warp] = runM;
                sh.wS[warp] = folded + s;   // relative to runOff = fp32(runM * c32)
            }
            workers_sync();
            float m = sh.wM[0];
            for (int w = 1; w < WARPS; ++w) m = fmaxf(m, sh.wM[w]);
            if (m > -CUDART_INF_F && m < CUDART_INF_F) {
                const double off = (double)__fmul_rn(m, c32);
                for (int w = 0; w < WARPS; ++w)
                    if (sh.wM[w] > -CUDART_INF_F) Z += sh.wS[w] * exp2((double)__fmul_rn(sh.wM[w], c32) - off);
                Z *= stream_sum_scale(m, c32);
            }
        }
        workers_sync();

        // ---- final selection and order --------------------------------------------------------
        int count = sh.count;
        workers_sync();
        if (count > k_eff) {
            keep_top_k<LOGIT16>(cand, keep, count, k_eff, sh);
            count = k_eff;
        }
        int n2 = 1;
        while (n2 < k_eff) n2 <<= 1;
        for (int i = tid; i < n2; i += THREADS) keep[i] = i < count ? cand[i] : 0ull;
        bitonic_sort_desc(keep, n2);

        const float top = key_logit(keep[0]);
        const bool bad = sh.nan || !(top > -CUDART_INF_F) || !(top < CUDART_INF_F) || (STATS && !(Z > 0.0));
        if (bad) {
            emit_invalid_row(a, row);
            if (tid == 0) atomicOr(a.status, ST_LOGIT);
            continue;
        }
        finish_row<false>(a, row, keep, k_eff, Tb, Z, sh);
    }
}

// Double-precision redo of the top-p cut for the rows in the queue, in one kernel: the exact chunk
// sums of the queued rows (four warps per chunk, two chunks per CTA at a time, the whole grid sharing
// the work) and, by the CTA that completes a row's last chunk, the cut of that row -- the sorted
// candidates are read back from q_idx, the exact normaliser is the sum of the row's chunk sums.
// Nothing waits (fence, then ticket); with an empty queue every CTA returns at once.
template <typename T>
__global__ void __launch_bounds__(THREADS) compress_precise_kernel(CompressArgs a, PreciseArgs p) {
    grid_dependency_sync();
    extern __shared__ u64 smem64[];
    u64* keep = smem64;
    __shared__ CompressShared sh;
    __shared__ double part[WARPS];
    __shared__ int last_slot[2];
    const int nq = *a.queue_count;
    if (nq == 0) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = warp >> 2, quarter = warp & 3;
    int k_eff = a.top_k > 0 ? a.top_k : a.k_max;
    if (k_eff > a.k_max) k_eff = a.k_max;
    if (k_eff > a.V) k_eff = a.V;
    const long long total = (long long)nq * a.nch;
    const long long pairs = (total + 1) / 2;
    for (long long pi = blockIdx.x; pi < pairs; pi += gridDim.x) {
        const long long item = 2 * pi + sub;
        int qslot = -1;
        const double s = precise_item_sum<T>(p, item, total, quarter, lane, qslot);
        if (lane == 0) part[warp] = s;
        __syncthreads();
        if (quarter == 0 && lane == 0) {
            int mine = -1;
            if (item < total) {
                precise_item_store(p, item, (part[warp] + part[warp + 1]) + (part[warp + 2] + part[warp + 3]));
                __threadfence();
                if (atomicAdd(&a.tickets[qslot], 1) == a.nch - 1) mine = qslot;
            }
            last_slot[sub] = mine;
        }
        __syncthreads();
        const int l0 = last_slot[0], l1 = last_slot[1];
        for (int which = 0; which < 2; ++which) {
            const int slot = which ? l1 : l0;
            if (slot < 0) continue;
            __threadfence();
            const int row = a.queue[slot];
            const int b = row / a.G;
            const T* rowp = reinterpret_cast<const T*>(a.logits) + (long long)row * a.row_stride;
            workers_sync();
            for (int j = tid; j < k_eff; j += THREADS) {
                const int v = a.q_idx[(long long)row * a.k_max + j];
                keep[j] = make_key(load_logit(rowp, v), v);
            }
            double z = 0.0;
            for (int c = tid; c < a.nch; c += THREADS) z += a.dsum[(long long)row * a.nch + c];
            z = warp_sum(z);
            if (lane == 0) sh.wS[warp] = z;
            workers_sync();
            double Z = 0.0;
            for (int w = 0; w < WARPS; ++w) Z += sh.wS[w];
            workers_sync();
            finish_row<true>(a, row, keep, k_eff, a.temperature[b], Z, sh);
        }
        __syncthreads();
    }
}

}  // namespace picospec
