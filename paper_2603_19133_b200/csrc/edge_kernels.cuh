// Edge-side correction of the paper's own data flow (Sec. 3.3): the verifier has sent the K
// largest components of the target distribution at the rejected position; the edge draws the
// corrected token from norm(max(0, P~ - Q)) against its own dense distribution Q.  Only the K
// transmitted indices can carry weight, so after the streaming statistics pass over the edge's row
// (the shared chunk-statistics kernels, which give the normaliser of Q) the work is O(K) per
// sequence: one CTA each.
#pragma once
#include "verify_kernels.cuh"

namespace picospec {

// Uses the fields of VerifyArgs as follows: logits = the edge's logits [B, G+1 rows per sequence,
// V]; pos [B] = the row; q_idx / q_prob [B, k_max] and q_count [B] = the transmitted components
// (one sparse row per sequence); u_resample [B] = one uniform per sequence; token [B]; mass [B].
template <typename T, bool PRECISE>
__global__ void __launch_bounds__(THREADS) edge_finish_kernel(VerifyArgs a) {
    grid_dependency_sync();
    __shared__ double warp_tot[WARPS];
    __shared__ double sZ, sZraw;
    __shared__ float smx;
    __shared__ int sbad, sfirst, slast, sflag;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G1 = a.G + 1;
    const int nloop = PRECISE ? *a.queue_count : a.B;
    for (int slot = blockIdx.x; slot < nloop; slot += gridDim.x) {
        const int b = PRECISE ? a.queue[slot] : slot;
        const float Tb = a.temperature[b];
        const float c32 = temp_scale(Tb);
        const int j = a.pos[b];
        const int n = a.q_count[b];
        unsigned st_bits = 0;
        if (!temp_ok(Tb)) st_bits |= ST_TEMPERATURE;
        if (j < 0 || j > a.G || n <= 0 || n > a.k_max) st_bits |= ST_RANGE;
        if (*(volatile unsigned*)a.status & ST_INTERNAL) st_bits |= ST_INTERNAL;   // incomplete statistics
        __syncthreads();
        if (tid == 0) {
            sbad = 0;
            sflag = 0;
            sfirst = 0x7fffffff;
            slast = -1;
        }
        __syncthreads();
        if (!st_bits && warp == 0) {
            double Z, Zraw;
            float mx;
            bool bad;
            row_stats<T>(a, b * G1 + j, c32, lane, PRECISE, Z, Zraw, mx, bad);
            if (lane == 0) {
                sZ = Z;
                sZraw = Zraw;
                smx = mx;
                if (!PRECISE) a.row_max[b * G1 + j] = mx;
                if (bad) sbad = (int)ST_LOGIT;
            }
        }
        __syncthreads();
        st_bits |= (unsigned)sbad;
        int token = -1;
        double R = -1.0;
        if (!st_bits) {
            const T* row = reinterpret_cast<const T*>(a.logits) + (long long)(b * G1 + j) * a.row_stride;
            const int* idx = a.q_idx + (long long)b * a.k_max;
            const float* prob = a.q_prob + (long long)b * a.k_max;
            Weight<PRECISE> wt;
            wt.init(Tb, smx);
            const double Z = sZ;
            // four consecutive stored entries per thread: index loads, then the logit gathers
            int vv[4];
            float pp[4], ll[4];
            bool rb = false;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int t = tid * 4 + e;
                vv[e] = t < n ? idx[t] : -2;
                pp[e] = t < n ? prob[t] : 0.f;
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool ok = vv[e] >= 0 && vv[e] < a.V;
                if (vv[e] != -2 && !ok) rb = true;
                ll[e] = ok ? load_logit(row, vv[e]) : -CUDART_INF_F;
            }
            if (rb) atomicOr(&sbad, (int)ST_RANGE);
            double r[4], cum[4], loc = 0.0, qloc = 0.0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool ok = vv[e] >= 0 && vv[e] < a.V;
                const double q = ok ? wt(ll[e]) / Z : 0.0;
                const double d = (double)pp[e] - q;
                r[e] = (ok && d > 0.0) ? d : 0.0;
                qloc += q;
                loc += r[e];
                cum[e] = loc;
            }
            double Rres, Q;
            double base = block_scan_incl(loc, warp_tot, Rres) - loc;
            block_scan_incl(qloc, warp_tot, Q);
            st_bits |= (unsigned)sbad;
            // every q carries a relative error of at most GUARD_Z in the fast path, so every prefix
            // and the total are off by at most GUARD_Z * Q
            const double E = PRECISE ? 0.0 : 2.0 * GUARD_Z * Q;
            // residual total too close to zero to say whether the fallback applies, or so small that the
            // normaliser's error would show in the reported mass: decide and report in double
            if (!PRECISE && (Rres <= E || Rres < RESID_EXACT_BELOW * Q) && tid == 0) sflag = 1;
            const bool fallback = !(Rres > E);
            if (fallback) {
                // Q covers every transmitted component: draw from the components themselves
                loc = 0.0;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    r[e] = (vv[e] >= 0 && vv[e] < a.V) ? (double)pp[e] : 0.0;
                    loc += r[e];
                    cum[e] = loc;
                }
                base = block_scan_incl(loc, warp_tot, Rres) - loc;
            }
            R = Rres;
            const double thr = (double)a.u_resample[b] * R;
            int mine = 0x7fffffff, mylast = -1;
#pragma unroll
            for (int e = 3; e >= 0; --e) {
                if (tid * 4 + e < n && base + cum[e] > thr) mine = tid * 4 + e;
                if (r[e] > 0.0 && mylast < 0) mylast = tid * 4 + e;
            }
            if (mine != 0x7fffffff) atomicMin(&sfirst, mine);
            if (mylast >= 0) atomicMax(&slast, mylast);
            __syncthreads();
            const int pick = sfirst != 0x7fffffff ? sfirst : slast;
            if (!PRECISE && !fallback) {
                if (sfirst == 0x7fffffff) {
                    if (tid == 0) sflag = 1;
                } else if (mine == sfirst) {
                    const int e = mine - tid * 4;
                    const double hi = base + cum[e] - thr;
                    const double lo = thr - (base + cum[e] - r[e]);
                    if (hi < E || (mine > 0 && lo < E)) sflag = 1;
                }
            }
            __syncthreads();
            if (pick >= 0) token = idx[pick];
        }
        if (tid == 0) {
            if (st_bits) {
                atomicOr(a.status, st_bits);
                a.token[b] = -1;
                if (a.mass) a.mass[b] = -1.f;
            } else {
                a.token[b] = token;
                if (a.mass) a.mass[b] = (float)R;
                if (!PRECISE && sflag) {
                    a.need_rows[b] = ~0ull;
                    a.queue[atomicAdd(a.queue_count, 1)] = b;
                    a.rowq[atomicAdd(a.rowq_count, 1)] = b * G1 + j;
                    atomicAdd(a.slow_rows, 1ull);
                }
            }
        }
    }
}

}  // namespace picospec
