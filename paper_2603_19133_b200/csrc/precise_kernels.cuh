// Double-precision chunk sums for rows whose fp32 statistics were too close to a decision
// threshold.  One warp per (queued row, chunk): sum of exp(l/T - max/T) over the chunk, exactly
// the terms of the definition.  The whole grid shares the work, so a handful of flagged rows
// costs microseconds; with an empty queue every CTA returns at once.
#pragma once
#include "common.cuh"

namespace picospec {

struct PreciseArgs {
    const void* logits;
    long long row_stride;
    int V, nch;
    int seq_rows;              // rows per sequence in the logits tensor (G or G+1)
    int expand;                // rows per queue entry: entry e covers rows e*expand .. +expand-1
    const int* pos;            // optional: entry b covers the single row b*seq_rows + pos[b]
    const float* temperature;  // [B]
    const int* queue;
    const int* queue_count;
    const unsigned long long* need_rows;   // optional [entries]: bit ri = row ri of the entry is wanted
    // optional row window of an entry: rows outside [r0, r1), or beyond gamma[entry], are never read
    int r0 = 0, r1 = 0x7fffffff;
    const int* gamma = nullptr;
    const float* row_max;      // [rows] exact row maxima from the fp32 pass
    double* dsum;              // [rows, nch]
};

template <typename T>
__global__ void __launch_bounds__(THREADS) precise_chunk_sums_kernel(PreciseArgs a) {
    grid_dependency_sync();
    const int nq = *a.queue_count;
    if (nq == 0) return;
    const int lane = threadIdx.x & 31;
    const long long gw = (long long)blockIdx.x * WARPS + (threadIdx.x >> 5);
    const long long nw = (long long)gridDim.x * WARPS;
    const long long total = (long long)nq * a.expand * a.nch;
    for (long long item = gw; item < total; item += nw) {
        const int c = (int)(item % a.nch);
        const long long t = item / a.nch;
        const int ri = (int)(t % a.expand);
        const int e = a.queue[(int)(t / a.expand)];
        if (a.need_rows && !a.pos && ri < 64 && !((a.need_rows[e] >> ri) & 1ull)) continue;
        if (!a.pos && (ri < a.r0 || ri >= a.r1 || (a.gamma && ri > a.gamma[e]))) continue;
        const int src_row = a.pos ? e * a.seq_rows + a.pos[e] : e * a.expand + ri;
        const int b = src_row / a.seq_rows;
        const T* row = reinterpret_cast<const T*>(a.logits) + (long long)src_row * a.row_stride;
        // x = l * (1/T) instead of l / T: one rounding of 2^-53 more per term, far below every
        // threshold this pass decides; four independent sums keep the exp pipeline busy
        const double rT = 1.0 / (double)a.temperature[b];
        const double m = (double)a.row_max[src_row] * rT;
        const int v0 = c * CHUNK;
        double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
#pragma unroll 2
        for (int k = lane; k < CHUNK; k += 128) {
            const int v = v0 + k;
            float l0 = -CUDART_INF_F, l1 = -CUDART_INF_F, l2 = -CUDART_INF_F, l3 = -CUDART_INF_F;
            if (v < a.V) l0 = load_logit(row, v);
            if (v + 32 < a.V) l1 = load_logit(row, v + 32);
            if (v + 64 < a.V) l2 = load_logit(row, v + 64);
            if (v + 96 < a.V) l3 = load_logit(row, v + 96);
            s0 += exp((double)l0 * rT - m);
            s1 += exp((double)l1 * rT - m);
            s2 += exp((double)l2 * rT - m);
            s3 += exp((double)l3 * rT - m);
        }
        double s = (s0 + s1) + (s2 + s3);
        s = warp_sum(s);
        if (lane == 0) a.dsum[(long long)src_row * a.nch + c] = s;
    }
}

}  // namespace picospec
