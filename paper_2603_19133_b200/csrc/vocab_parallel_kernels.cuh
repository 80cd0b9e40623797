// Vocabulary-parallel verification: the small kernels around the shared ones.
//
// The verifier model of the paper runs on two to four GPUs (Sec. 4.1), so its output layer leaves
// the target logits sharded along the vocabulary: rank r holds the columns [v0, v0 + Vs) of every
// row, v0 a multiple of the 1024-entry chunk, every rank but the last the same number of chunks.
// One verification is then
//   1. per rank, on its slice: the streaming statistics pass (chunk records) and vp_gather_kernel
//      (the logits at the stored entries and drafted tokens the slice holds, -inf for the others);
//   2. exchange: all-gather of the records, element-wise maximum of the gathered logits;
//   3. every rank: the finish kernel on the exchanged arrays (accept test, residual masses, scan,
//      level-1 pick of a chunk), which leaves the draw to the chunk's owner;
//   4. the owner: vp_draw_kernel (level 2 inside the chunk, from its slice); element-wise maximum
//      of tokens and of the owners' "too close to call" flags;
//   5. vp_queue_kernel builds the list of sequences for the double-precision pass from the flags of
//      steps 3 and 4 (the same list on every rank); that pass repeats 1 - 4 with exact chunk sums
//      of the listed rows, and vp_merge_kernel puts its tokens in place.
// The exchanges are the caller's (NCCL all-gather / all-reduce, or plain copies when the slices
// live in one memory); nothing here touches another rank's memory.
#pragma once
#include "verify_kernels.cuh"

namespace picospec {

// Logits of this slice at the stored entries (slots 0 .. k_max - 1) and at the drafted token (slot
// k_max) of every draft position; -inf where the index lies outside the slice, the slot is beyond
// the row's count, or the index is out of range.
template <typename T>
__global__ void __launch_bounds__(THREADS) vp_gather_kernel(VerifyArgs a, int v0, int Vs, float* entries) {
    grid_dependency_sync();
    const int G = a.G, G1 = a.G + 1, K1 = a.k_max + 1;
    const long long total = (long long)a.B * G * K1;
    for (long long e = (long long)blockIdx.x * THREADS + threadIdx.x; e < total; e += (long long)gridDim.x * THREADS) {
        const int ri = (int)(e / K1), k = (int)(e - (long long)ri * K1);
        const int b = ri / G, i = ri - b * G;
        int v = -1;
        if (k == a.k_max) {
            v = a.draft_tok[ri];
        } else {
            const int n = a.q_count[ri];
            if (k < n && n <= a.k_max) v = a.q_idx[(long long)ri * a.k_max + k];
        }
        float l = -CUDART_INF_F;
        if (v >= v0 && v < v0 + Vs) {
            const T* row = reinterpret_cast<const T*>(a.logits) + (long long)(b * G1 + i) * a.row_stride;
            l = load_logit(row, v - v0);
        }
        entries[e] = l;
    }
}

// The draw inside the picked chunk, by the rank that owns it: one CTA per sequence.  a.logits is the
// slice (columns v0 ..), a.V the size of the whole vocabulary; a.pick comes from the finish kernel;
// listed (or null: every sequence) marks the sequences of the double-precision pass.  tok_flag [2, B]:
// the token, or -1 where another rank owns the chunk or there is nothing to draw; and 1 where the
// fast pass could not call the draw.
template <typename T, bool PRECISE>
__global__ void __launch_bounds__(THREADS) vp_draw_kernel(VerifyArgs a, int v0, int my_rank, const int* listed, int* tok_flag) {
    __shared__ FinishShared sh;
    __shared__ double sZ;
    __shared__ float smx;
    __shared__ int sbad;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = a.G, G1 = a.G + 1;
    grid_dependency_sync();
    for (int b = blockIdx.x; b < a.B; b += gridDim.x) {
        __syncthreads();
        int token = -1;
        const int j = a.pick[4 * b + 0], cs = a.pick[4 * b + 1], fl = a.pick[4 * b + 2];
        const int L = a.chunks_per_rank > 0 ? a.chunks_per_rank : a.nch;
        const bool mine = cs >= 0 && cs < a.nch && cs / L == my_rank && j >= 0 && j <= G && (!PRECISE || !listed || listed[b] == 1);
        if (tid == 0) {
            sh.flag = 0;
            sbad = 0;
        }
        __syncthreads();
        if (mine) {
            const float Tb = a.temperature[b];
            const float c32 = temp_scale(Tb);
            if (warp == 0) {
                double Z, Zraw;
                float mx;
                bool bad;
                const unsigned long long need = PRECISE ? a.need_rows[b] : 0ull;
                row_stats<T>(a, b * G1 + j, c32, lane, PRECISE && row_needed(need, j), Z, Zraw, mx, bad);
                if (lane == 0) {
                    sZ = Z;
                    smx = mx;
                    sbad = bad || !temp_ok(Tb);
                }
            }
            __syncthreads();
            if (!sbad) {
                const bool use_resid = (fl & PICK_RESIDUAL) != 0 && j < G;
                const int rj = b * G + (j < G ? j : 0);
                int n = use_resid ? a.q_count[rj] : 0;
                if (n < 0 || n > a.k_max) n = 0;
                Weight<PRECISE> wt;
                wt.init(Tb, smx);
                const T* row = reinterpret_cast<const T*>(a.logits) + (long long)(b * G1 + j) * a.row_stride;
                token = level2_draw<T, PRECISE>(a, row, v0, cs, a.q_idx + (long long)rj * a.k_max,
                                                a.q_prob + (long long)rj * a.k_max, n, use_resid && n > 0, wt, 1.0 / sZ,
                                                a.u_resample[2 * b + 1], sh);
            }
        }
        if (tid == 0) {
            tok_flag[b] = token;
            tok_flag[a.B + b] = (!PRECISE && mine && sh.flag) ? 1 : 0;
        }
    }
}

// After the exchange of the fast pass's tokens and flags: the tokens of the sequences that are
// final, and the list of those that take the double-precision pass (sequence order, so every rank
// builds the same list).  One CTA.  listed[b]: 0 = final, 1 = redone, 2 = only small residual
// masses are recomputed.
__global__ void __launch_bounds__(THREADS) vp_queue_kernel(VerifyArgs a, const int* tok_flag, int* listed) {
    __shared__ int warp_tot[WARPS];
    __shared__ int carry;
    grid_dependency_sync();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) carry = 0;
    __syncthreads();
    unsigned long long rows = 0ull;
    for (int b0 = 0; b0 < a.B; b0 += THREADS) {
        const int b = b0 + tid;
        int kind = 0, entry = 0;
        if (b < a.B) {
            const int fl = a.pick[4 * b + 2];
            const bool l2 = tok_flag[a.B + b] != 0;
            if ((fl & PICK_FLAGGED) || l2) {
                const bool mass_only = (fl & PICK_MASS_ONLY) && !l2;
                kind = mass_only ? 2 : 1;
                entry = b | ((fl & PICK_DRAW_ONLY) ? QUEUE_DRAW_ONLY : 0) | (mass_only ? QUEUE_MASS_ONLY : 0);
                rows += (unsigned long long)a.pick[4 * b + 3];
            }
            listed[b] = kind;
            if (a.token) a.token[b] = tok_flag[b];
        }
        const int one = kind ? 1 : 0;
        int incl = one;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += y;
        }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        int base = carry;
        for (int w = 0; w < warp; ++w) base += warp_tot[w];
        if (kind) a.queue[base + incl - 1] = entry;
        __syncthreads();
        if (tid == THREADS - 1) carry = base + incl;
        __syncthreads();
    }
    if (rows) atomicAdd(a.slow_rows, rows);
    if (tid == 0) {
        *a.queue_count = carry;
        *a.rowq_count = 0;
    }
    __syncthreads();
    // the rows of the listed sequences that need exact chunk sums (any order: every rank sums its
    // own slice of each, and the results are exchanged as whole arrays)
    const int G1 = a.G + 1;
    for (int b = tid; b < a.B; b += THREADS) {
        if (!listed[b]) continue;
        const unsigned long long nd = a.need_rows[b];
        for (int i = 0; i < G1; ++i)
            if (i >= 64 || ((nd >> i) & 1ull)) a.rowq[atomicAdd(a.rowq_count, 1)] = b * G1 + i;
    }
}

// After the exchange of the double-precision pass's tokens: they replace the fast ones.
__global__ void __launch_bounds__(THREADS) vp_merge_kernel(int B, const int* listed, const int* tok_flag, int* token) {
    grid_dependency_sync();
    for (int b = blockIdx.x * THREADS + threadIdx.x; b < B; b += gridDim.x * THREADS)
        if (listed[b] == 1) token[b] = tok_flag[b];
}

}  // namespace picospec
