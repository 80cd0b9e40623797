// Wire format of the sparse rows (Sec. 3.3: the verifier sends pairs of vocabulary id and
// probability -- under 100 bytes for K = 10 -- laid out so that the receiver can view the arrays in place).  One message:
//     0   u32  magic 0x31505350 ("PSP1")
//     4   u32  R, the number of rows
//     8   u16  K, the capacity of a dense row
//     10  u16  probability type: 0 = fp32, 1 = fp16 (round to nearest even)
//     12  u32  N = sum over rows of max(count, 0)
//     16  i16  count[R]   (-1 = invalid row), zero-padded to a multiple of 4 bytes
//     ..  i32  id[N]      rows in order, entries in stored order
//     ..  prob[N]         fp32 or fp16; the message is zero-padded to a multiple of 4 bytes
// Packing and unpacking are two small kernels each: an exclusive scan of the counts by one CTA,
// then one warp per row moving its entries.
#pragma once
#include <cuda_fp16.h>

#include "common.cuh"

namespace picospec {

constexpr unsigned WIRE_MAGIC = 0x31505350u;

struct WireArgs {
    int* q_idx;                 // [R, K]   (read by pack, written by unpack)
    float* q_prob;              // [R, K]
    int* q_count;               // [R]
    int R, K, prob_type;
    unsigned char* buf;         // the message
    long long capacity;         // bytes available at buf (pack) / bytes of the message (unpack)
    long long* bytes_out;       // pack: size of the message, or -1 if it does not fit
    int* offsets;               // workspace [R + 1]: first entry of each row; [R] = N, or -1 = refused
    unsigned* status;
};

__host__ __device__ __forceinline__ long long wire_pad4(long long n) { return (n + 3) / 4 * 4; }
__host__ __device__ __forceinline__ long long wire_bytes(long long rows, long long entries, int prob_type) {
    return 16 + wire_pad4(2 * rows) + 4 * entries + wire_pad4((prob_type == 0 ? 4 : 2) * entries);
}

// One CTA: exclusive scan of max(count, 0) over the rows; then the header (pack: only once the
// message is known to fit the caller's buffer, so that a buffer that is too small is never written),
// or the header and count checks (unpack).  The packed counts are written by the move kernel.
template <bool PACK>
__global__ void __launch_bounds__(THREADS) wire_scan_kernel(WireArgs a) {
    __shared__ int warp_tot[WARPS];
    __shared__ int carry_s, bad_s;
    grid_dependency_sync();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        carry_s = 0;
        bad_s = 0;
    }
    __syncthreads();
    const short* wire_counts = reinterpret_cast<const short*>(a.buf + 16);
    if (!PACK && tid == 0) {
        // header: refuse a message for another shape, of another kind, or cut short
        bool ok = a.capacity >= 16;
        if (ok) {
            const unsigned* h = reinterpret_cast<const unsigned*>(a.buf);
            const unsigned k = h[2] & 0xffffu, pt = h[2] >> 16;
            ok = h[0] == WIRE_MAGIC && h[1] == (unsigned)a.R && k == (unsigned)a.K && pt <= 1u &&
                 a.capacity >= wire_bytes(a.R, h[3], (int)pt);
        }
        if (!ok) bad_s = 1;
    }
    __syncthreads();
    const bool refused = !PACK && bad_s;
    for (int r0 = 0; r0 < a.R && !refused; r0 += THREADS) {
        const int r = r0 + tid;
        int c = 0;
        if (r < a.R) {
            c = PACK ? a.q_count[r] : (int)wire_counts[r];
            if (c > a.K || c < -1) {
                bad_s = 1;          // pack: the row travels as invalid; unpack: the message is refused
                c = -1;
            }
        }
        const int n = c > 0 ? c : 0;
        int incl = n;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += y;
        }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        int base = carry_s;
        for (int w = 0; w < warp; ++w) base += warp_tot[w];
        if (r < a.R) a.offsets[r] = base + incl - n;
        __syncthreads();
        if (tid == THREADS - 1) carry_s = base + incl;
        __syncthreads();
    }
    if (tid == 0) {
        const int N = carry_s;
        if (PACK) {
            const long long need = wire_bytes(a.R, N, a.prob_type);
            const bool fits = need <= a.capacity;
            a.offsets[a.R] = fits ? N : -1;
            *a.bytes_out = fits ? need : -1;
            if (bad_s) atomicOr(a.status, ST_RANGE);
            if (fits) {
                unsigned* h = reinterpret_cast<unsigned*>(a.buf);
                h[0] = WIRE_MAGIC;
                h[1] = (unsigned)a.R;
                h[2] = (unsigned)a.K | ((unsigned)a.prob_type << 16);
                h[3] = (unsigned)N;
                if (a.R & 1) reinterpret_cast<short*>(a.buf + 16)[a.R] = 0;      // padding of the counts
                if (a.prob_type == 1 && (N & 1))                                  // padding of the message
                    *reinterpret_cast<unsigned short*>(a.buf + need - 2) = 0;
            } else {
                atomicOr(a.status, ST_RANGE);
            }
        } else {
            bool ok = !bad_s;
            if (ok) ok = (unsigned)N == reinterpret_cast<const unsigned*>(a.buf)[3];
            a.offsets[a.R] = ok ? N : -1;
            if (!ok) atomicOr(a.status, ST_RANGE);
        }
    }
}

// One warp per row.
template <bool PACK>
__global__ void __launch_bounds__(THREADS) wire_move_kernel(WireArgs a) {
    grid_dependency_sync();
    const int lane = threadIdx.x & 31;
    const int N = a.offsets[a.R];
    const int ptype = PACK ? a.prob_type : (N >= 0 ? (int)(reinterpret_cast<const unsigned*>(a.buf)[2] >> 16) : 0);
    int* ids = reinterpret_cast<int*>(a.buf + 16 + wire_pad4(2ll * a.R));
    unsigned char* probs = reinterpret_cast<unsigned char*>(ids + (N > 0 ? N : 0));
    for (int r = blockIdx.x * WARPS + (threadIdx.x >> 5); r < a.R; r += gridDim.x * WARPS) {
        int* qi = a.q_idx + (long long)r * a.K;
        float* qp = a.q_prob + (long long)r * a.K;
        if (PACK) {
            if (N < 0) continue;                              // the message did not fit: nothing is written
            int c = a.q_count[r];
            if (c > a.K || c < -1) c = -1;                    // the row travels as invalid
            const int n = c > 0 ? c : 0;
            const int o = a.offsets[r];
            if (lane == 0) reinterpret_cast<short*>(a.buf + 16)[r] = (short)c;
            for (int j = lane; j < n; j += 32) {
                ids[o + j] = qi[j];
                if (ptype == 0) reinterpret_cast<float*>(probs)[o + j] = qp[j];
                else reinterpret_cast<__half*>(probs)[o + j] = __float2half_rn(qp[j]);
            }
        } else {
            const int c = N < 0 ? -1 : (int)reinterpret_cast<const short*>(a.buf + 16)[r];
            const int n = c > 0 ? c : 0;
            const int o = N < 0 ? 0 : a.offsets[r];
            for (int j = lane; j < a.K; j += 32) {
                int id = -1;
                float p = 0.f;
                if (j < n) {
                    id = ids[o + j];
                    p = ptype == 0 ? reinterpret_cast<const float*>(probs)[o + j]
                                   : __half2float(reinterpret_cast<const __half*>(probs)[o + j]);
                }
                qi[j] = id;
                qp[j] = p;
            }
            if (lane == 0) a.q_count[r] = c;
        }
    }
}

}  // namespace picospec
