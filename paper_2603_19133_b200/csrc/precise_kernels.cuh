// Double-precision chunk sums for rows whose fp32 statistics were too close to a decision
// threshold.  Four warps per (listed row, chunk): sum of exp(l/T - max/T) over the chunk, exactly
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
    const float* temperature;  // [B]
    const int* rows;           // the rows whose exact chunk sums are wanted (indices into the logits tensor)
    const int* row_count;      // how many
    const float* row_max;      // [rows] exact row maxima from the fp32 pass
    double* dsum;              // [rows, pitch]
    int pitch = 0;             // chunk sums per row in dsum (0: nch)
};

// One quarter of one item of the double-precision pass, by one warp.  Item = (listed row, chunk);
// returns the partial sum and the position of the row in the list.
template <typename T>
__device__ __forceinline__ double precise_item_sum(const PreciseArgs& a, long long item, long long total, int quarter,
                                                   int lane, int& qslot) {
    qslot = -1;
    double s = 0.0;
    if (item < total) {
        const int c = (int)(item % a.nch);
        qslot = (int)(item / a.nch);
        const int src_row = a.rows[qslot] & 0x1FFFFFFF;     // (a list may keep flags above the index)
        const int b = src_row / a.seq_rows;
        const T* row = reinterpret_cast<const T*>(a.logits) + (long long)src_row * a.row_stride;
        // x = l * (1/T) instead of l / T: one rounding of 2^-53 more per term, far below every
        // threshold this pass decides; four independent sums keep the exp pipeline busy
        const double rT = 1.0 / (double)a.temperature[b];
        const double m = (double)a.row_max[src_row] * rT;
        const int v0 = c * CHUNK + quarter * (CHUNK / 4);
        double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
#pragma unroll
        for (int k = lane; k < CHUNK / 4; k += 128) {
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
        s = warp_sum((s0 + s1) + (s2 + s3));
    }
    return s;
}
// where the sum of an item goes
__device__ __forceinline__ void precise_item_store(const PreciseArgs& a, long long item, double sum) {
    const int c = (int)(item % a.nch);
    const int src_row = a.rows[(int)(item / a.nch)] & 0x1FFFFFFF;
    a.dsum[(long long)src_row * (a.pitch > 0 ? a.pitch : a.nch) + c] = sum;
}

template <typename T>
__global__ void __launch_bounds__(THREADS) precise_chunk_sums_kernel(PreciseArgs a) {
    grid_dependency_sync();
    const int nq = *a.row_count;
    if (nq == 0) return;
    // A CTA takes two chunks at a time, four warps per chunk (a quarter of the chunk each, so that a
    // handful of rows still spreads over the whole GPU); the four partial sums of a chunk are added in
    // a fixed order.
    __shared__ double part[WARPS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = warp >> 2, quarter = warp & 3;
    const long long total = (long long)nq * a.nch;
    const long long pairs = (total + 1) / 2;
    for (long long pi = blockIdx.x; pi < pairs; pi += gridDim.x) {
        const long long item = 2 * pi + sub;
        int qslot;
        const double s = precise_item_sum<T>(a, item, total, quarter, lane, qslot);
        if (lane == 0) part[warp] = s;
        __syncthreads();
        if (item < total && quarter == 0 && lane == 0)
            precise_item_store(a, item, (part[warp] + part[warp + 1]) + (part[warp + 2] + part[warp + 3]));
        __syncthreads();
    }
}

}  // namespace picospec
