// Shared device helpers of the picospec kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

namespace picospec {

constexpr int CHUNK = 1024;        // vocabulary entries per level-1 chunk (sampler definition)
constexpr int THREADS = 256;       // threads per CTA in every kernel of the library
constexpr int WARPS = THREADS / 32;
constexpr int MAX_G1 = 65;         // gamma + 1 <= 65
constexpr int MAX_K = 1024;        // capacity limit of a sparse row

// Bound on the relative error of an fp32-accumulated normaliser / chunk mass against exact
// arithmetic on the same inputs: ex2.approx (2^-22), one fma rounding of the exponent argument
// and the fp32 rounding of log2(e)/T, both weighted by the mass-averaged |log2(w_v/w_max)| <=
// log2(V) ~ 18 bits, plus accumulation rounding.  Sum ~2e-6; decisions closer than this to
// their threshold are re-taken in double precision.
constexpr double GUARD_Z = 3e-6;
constexpr double BORDER_REL = 1e-6;   // "borderline" band of the accept test
// A residual mass R = 1 - sum min(p, q~) carries the absolute error of the fp32-accumulated
// normaliser (a few 1e-7 in practice, GUARD_Z at worst); below this value it would miss the 1e-5
// relative target, so such a position is recomputed from the exact chunk sums.
constexpr double RESID_EXACT_BELOW = 0.05;
// The residual norm(max(0, p - q~)) is undefined when max(0, p - q~) vanishes; the draw is then from
// p itself.  The verify path forms chunk masses of the residual as (chunk mass of p) - sum min(p, q~),
// which in double precision cannot tell a mass of 1e-16 from zero: a residual whose total mass
// (of a row that sums to one) is at most this value counts as vanished.
constexpr double RESID_ZERO_BELOW = 1e-12;

// device status bits (mirrors picospec.h)
constexpr unsigned ST_TEMPERATURE = 1u, ST_LOGIT = 2u, ST_RANGE = 4u;

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// log2(e) / T in fp32, round-to-nearest: the one scale every fp32 pass and its double-precision
// epilogue agree on.
__device__ __forceinline__ float temp_scale(float T) { return __fdiv_rn(1.4426950408889634f, T); }
__device__ __forceinline__ bool temp_ok(float T) { return T > 0.0f && T < CUDART_INF_F; }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, d));
    return v;
}
// maximum over the warp in one instruction; NaN inputs are ignored (all NaN gives NaN)
__device__ __forceinline__ float warp_max_redux(float v) {
    float r;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}

// Barrier over the 256 worker threads (warps 0..7) of a CTA.  Kernels that carry an extra producer
// warp cannot use __syncthreads in code their workers share with plain 256-thread kernels, so the
// cooperative routines below all synchronise on named barrier 1.
__device__ __forceinline__ void workers_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
// The same barrier, returning the OR of `pred` over the 256 workers.
__device__ __forceinline__ bool workers_sync_or(bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, 256, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)pred)
        : "memory");
    return r != 0;
}

// Inclusive scan of one double per thread over the 256 worker threads.  warp_tot: 8 doubles of
// shared memory.  Contains two barriers.
__device__ __forceinline__ double block_scan_incl(double x, double* warp_tot, double& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        double y = __shfl_up_sync(0xffffffffu, x, d);
        if (lane >= d) x += y;
    }
    if (lane == 31) warp_tot[warp] = x;
    workers_sync();
    double base = 0.0, tot = 0.0;
#pragma unroll
    for (int w = 0; w < WARPS; ++w) {
        double t = warp_tot[w];
        if (w < warp) base += t;
        tot += t;
    }
    workers_sync();
    total = tot;
    return x + base;
}

// ---- logits element access -------------------------------------------------------------

__device__ __forceinline__ float load_logit(const float* row, long long v) { return __ldg(row + v); }
__device__ __forceinline__ float load_logit(const __nv_bfloat16* row, long long v) {
    unsigned short h = __ldg(reinterpret_cast<const unsigned short*>(row) + v);
    return __uint_as_float(static_cast<uint32_t>(h) << 16);
}

__device__ __forceinline__ uint4 ld_stream_v4(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// One chunk of 1024 logits held by a warp: 32 values per lane.
//   bf16: 4 vectors of 8; lane's vector j covers v0 + j*256 + lane*8 .. +7, packed two per word
//   fp32: 8 vectors of 4; lane's vector j covers v0 + j*128 + lane*4 .. +3
// Entries at or beyond V read as -inf (weight zero, never a candidate).
template <typename T> struct ChunkRegs;

template <> struct ChunkRegs<__nv_bfloat16> {
    uint32_t w[16];
    static constexpr int VEC = 8, NVEC = 4;
    template <bool ALIGNED> __device__ __forceinline__ void load(const __nv_bfloat16* row, int v0, int V, int lane) {
#pragma unroll
        for (int j = 0; j < NVEC; ++j) {
            const int v = v0 + j * 256 + lane * 8;
            if (ALIGNED && v + 8 <= V) {
                uint4 q = ld_stream_v4(row + v);
                w[4 * j + 0] = q.x; w[4 * j + 1] = q.y; w[4 * j + 2] = q.z; w[4 * j + 3] = q.w;
            } else {
                const unsigned short* r16 = reinterpret_cast<const unsigned short*>(row);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    uint32_t lo = (v + 2 * e < V) ? __ldg(r16 + v + 2 * e) : 0xFF80u;
                    uint32_t hi = (v + 2 * e + 1 < V) ? __ldg(r16 + v + 2 * e + 1) : 0xFF80u;
                    w[4 * j + e] = lo | (hi << 16);
                }
            }
        }
    }
    // value k (0..31) of this lane and its vocabulary offset relative to v0
    __device__ __forceinline__ float value(int k) const {
        return (k & 1) ? __uint_as_float(w[k >> 1] & 0xffff0000u) : __uint_as_float(w[k >> 1] << 16);
    }
    static __device__ __forceinline__ int offset(int k, int lane) { return (k >> 3) * 256 + lane * 8 + (k & 7); }
    // maximum of vector j (8 values), NaN ignored
    __device__ __forceinline__ float vec_max(int j) const {
        __nv_bfloat162 m = *reinterpret_cast<const __nv_bfloat162*>(&w[4 * j]);
#pragma unroll
        for (int k = 1; k < 4; ++k) m = __hmax2(m, *reinterpret_cast<const __nv_bfloat162*>(&w[4 * j + k]));
        uint32_t mm = *reinterpret_cast<uint32_t*>(&m);
        return fmaxf(__uint_as_float(mm << 16), __uint_as_float(mm & 0xffff0000u));
    }
    // maximum of the lane's 32 values, NaN ignored
    __device__ __forceinline__ float lane_max_plain() const {
        __nv_bfloat162 m[8];
#pragma unroll
        for (int k = 0; k < 8; ++k)
            m[k] = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&w[2 * k]), *reinterpret_cast<const __nv_bfloat162*>(&w[2 * k + 1]));
#pragma unroll
        for (int k = 0; k < 4; ++k) m[k] = __hmax2(m[2 * k], m[2 * k + 1]);
        const __nv_bfloat162 a = __hmax2(__hmax2(m[0], m[1]), __hmax2(m[2], m[3]));
        const uint32_t mm = *reinterpret_cast<const uint32_t*>(&a);
        return fmaxf(__uint_as_float(mm << 16), __uint_as_float(mm & 0xffff0000u));
    }
    // NaN-propagating maximum of the lane's 32 values
    __device__ __forceinline__ float lane_max() const {
        __nv_bfloat162 m = *reinterpret_cast<const __nv_bfloat162*>(&w[0]);
#pragma unroll
        for (int k = 1; k < 16; ++k) m = __hmax2_nan(m, *reinterpret_cast<const __nv_bfloat162*>(&w[k]));
        uint32_t mm = *reinterpret_cast<uint32_t*>(&m);
        float lo = __uint_as_float(mm << 16), hi = __uint_as_float(mm & 0xffff0000u);
        return (lo != lo || hi != hi) ? CUDART_NAN_F : fmaxf(lo, hi);
    }
};

template <> struct ChunkRegs<float> {
    float f[32];
    static constexpr int VEC = 4, NVEC = 8;
    template <bool ALIGNED> __device__ __forceinline__ void load(const float* row, int v0, int V, int lane) {
#pragma unroll
        for (int j = 0; j < NVEC; ++j) {
            const int v = v0 + j * 128 + lane * 4;
            if (ALIGNED && v + 4 <= V) {
                uint4 q = ld_stream_v4(row + v);
                f[4 * j + 0] = __uint_as_float(q.x); f[4 * j + 1] = __uint_as_float(q.y);
                f[4 * j + 2] = __uint_as_float(q.z); f[4 * j + 3] = __uint_as_float(q.w);
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) f[4 * j + e] = (v + e < V) ? __ldg(row + v + e) : -CUDART_INF_F;
            }
        }
    }
    __device__ __forceinline__ float value(int k) const { return f[k]; }
    static __device__ __forceinline__ int offset(int k, int lane) { return (k >> 2) * 128 + lane * 4 + (k & 3); }
    __device__ __forceinline__ float vec_max(int j) const {
        return fmaxf(fmaxf(f[4 * j], f[4 * j + 1]), fmaxf(f[4 * j + 2], f[4 * j + 3]));
    }
    __device__ __forceinline__ float lane_max_plain() const {
        float m[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) m[k] = fmaxf(fmaxf(f[4 * k], f[4 * k + 1]), fmaxf(f[4 * k + 2], f[4 * k + 3]));
        return fmaxf(fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3])), fmaxf(fmaxf(m[4], m[5]), fmaxf(m[6], m[7])));
    }
    __device__ __forceinline__ float lane_max() const {
        float m = f[0];
        bool nan = f[0] != f[0];
#pragma unroll
        for (int k = 1; k < 32; ++k) {
            nan |= f[k] != f[k];
            m = fmaxf(m, f[k]);
        }
        return nan ? CUDART_NAN_F : m;
    }
};

// sum over the lane's 32 values of 2^(l * c - off) with the hardware ex2 (fp32)
template <typename T> __device__ __forceinline__ float lane_exp_sum(const ChunkRegs<T>& r, float c, float off) {
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
    for (int k = 0; k < 32; k += 4) {
        a0 += ex2_approx(fmaf(r.value(k + 0), c, -off));
        a1 += ex2_approx(fmaf(r.value(k + 1), c, -off));
        a2 += ex2_approx(fmaf(r.value(k + 2), c, -off));
        a3 += ex2_approx(fmaf(r.value(k + 3), c, -off));
    }
    return (a0 + a1) + (a2 + a3);
}

// Every kernel is launched with programmatic stream serialization: its CTAs may be scheduled while
// the kernel before it in the stream is still draining.  Each thread waits here, before its first
// access to global memory, until that kernel has completed and its writes are visible; then the
// CTA allows the kernel after it to be scheduled in the same way.  (Without the launch attribute
// both instructions do nothing.)
__device__ __forceinline__ void grid_dependency_sync() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Double-precision weight of one logit: exp(l * (1/T) - row_max * (1/T)) (the definition's
// exp(l/T - max/T) with the division replaced by one multiplication: 2^-53 relative per term).
// The fp32 streaming pass sums 2^(l*c32 - off) with c32 = fp32(log2 e / T) and
// off = fp32(row_max * c32); stream_sum_scale() is the exact factor 2^(off - row_max*c32) that
// brings such a sum onto the scale of these weights (what remains is the bounded error GUARD_Z).
// The fast path and the double-precision re-evaluation use the same weights; they differ in
// where the normaliser comes from.
template <bool PRECISE> struct Weight {
    double t, m;
    __device__ __forceinline__ void init(float T, float row_max) {
        t = 1.0 / (double)T;
        m = (double)row_max * t;
    }
    __device__ __forceinline__ double operator()(float l) const { return exp((double)l * t - m); }
};
__device__ __forceinline__ double stream_sum_scale(float row_max, float c32) {
    return exp2((double)__fmul_rn(row_max, c32) - (double)row_max * (double)c32);
}

}  // namespace picospec
