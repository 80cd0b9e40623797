// Shared-memory staging of logit rows with bulk asynchronous copies (cp.async.bulk) and
// mbarriers: one producer lane keeps STAGES tiles in flight, consumer warps take a tile as soon
// as its bytes have landed and hand the stage back once they have moved it to registers.
// Every wait is bounded: a barrier that does not complete within the limit makes the waiting
// warp record ST_INTERNAL in the status word and stop computing; it keeps consuming tiles (with the
// long limit) so that every copy that was issued has landed before its CTA exits.
#pragma once
#include "common.cuh"

namespace picospec {

constexpr unsigned ST_INTERNAL = 8u;          // a bounded wait ran out (mirrors picospec.h)
#ifndef PICOSPEC_WAIT_HINT_NS
#define PICOSPEC_WAIT_HINT_NS 20000u      // suspend-time hint of one mbarrier.try_wait
#endif
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // a wait gives up after two seconds

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
// makes the initialised barriers visible to the asynchronous proxy
__device__ __forceinline__ void mbar_init_fence() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// non-blocking: has the phase completed?
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// the same with a suspend-time hint (ns): the thread may sleep in hardware instead of polling
__device__ __forceinline__ bool mbar_try_wait_hint(uint64_t* bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity), "r"(ns)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// false: the time limit ran out
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, unsigned long long limit_ns) {
    // a limit of zero: only a wait that is complete already succeeds (try_wait may itself suspend the
    // thread for a while, so this case asks with the non-blocking test_wait)
    if (limit_ns == 0ull) return mbar_test_wait(bar, parity);
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t i = 1;; ++i) {
        if (mbar_try_wait_hint(bar, parity, PICOSPEC_WAIT_HINT_NS)) return true;
        if ((i & 7u) == 0u && global_ns() - t0 > limit_ns) return false;
    }
}
// The wait of the staged kernels, in two steps: first with the caller's limit, then -- so that no CTA
// leaves while a bulk copy into its shared memory is still in flight -- once more with the long limit.
//   WAIT_OK    completed within `limit_ns`;
//   WAIT_LATE  completed, but only after `limit_ns` had run out: the caller records ST_INTERNAL, stops
//              computing and keeps consuming, so every issued copy still lands and is waited for;
//   WAIT_LOST  not complete after the long limit either: the caller gives up for good.
enum { WAIT_OK = 0, WAIT_LATE = 1, WAIT_LOST = 2 };
__device__ __forceinline__ int mbar_wait_twice(uint64_t* bar, uint32_t parity, unsigned long long limit_ns) {
    if (mbar_wait(bar, parity, limit_ns)) return WAIT_OK;
    return mbar_wait(bar, parity, WAIT_LIMIT_NS) ? WAIT_LATE : WAIT_LOST;
}

__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

// Global -> shared bulk copy of `bytes` (a multiple of 16; both addresses 16-byte aligned) that
// reports its bytes to `bar`.
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar,
                                          uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_addr(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar)), "l"(policy)
        : "memory");
}

// ---- packed fp32 pairs (fma.rn.f32x2 / add.rn.f32x2) ------------------------------------------
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1,%2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
    asm("mov.b64 {%0,%1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 ffma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ f32x2 fadd2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// Sum over the lane's 32 values of 2^(l * c - off), two values per fma / add.  Each component is
// rounded exactly as the scalar fma / add would round it.
__device__ __forceinline__ float lane_exp_sum2(const ChunkRegs<__nv_bfloat16>& r, float c, float off) {
    const f32x2 C = pack2(c, c), O = pack2(-off, -off);
    f32x2 acc[4] = {pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f)};
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        const f32x2 x = pack2(__uint_as_float(r.w[k] << 16), __uint_as_float(r.w[k] & 0xffff0000u));
        float t0, t1;
        unpack2(ffma2(x, C, O), t0, t1);
        acc[k & 3] = fadd2(acc[k & 3], pack2(ex2_approx(t0), ex2_approx(t1)));
    }
    float a0, a1;
    unpack2(fadd2(fadd2(acc[0], acc[1]), fadd2(acc[2], acc[3])), a0, a1);
    return a0 + a1;
}
__device__ __forceinline__ float lane_exp_sum2(const ChunkRegs<float>& r, float c, float off) {
    const f32x2 C = pack2(c, c), O = pack2(-off, -off);
    f32x2 acc[4] = {pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f)};
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        float t0, t1;
        unpack2(ffma2(pack2(r.f[2 * k], r.f[2 * k + 1]), C, O), t0, t1);
        acc[k & 3] = fadd2(acc[k & 3], pack2(ex2_approx(t0), ex2_approx(t1)));
    }
    float a0, a1;
    unpack2(fadd2(fadd2(acc[0], acc[1]), fadd2(acc[2], acc[3])), a0, a1);
    return a0 + a1;
}

// ---- tile geometry ----------------------------------------------------------------------------
constexpr int TILE_CHUNKS = WARPS;               // one chunk per consumer warp
constexpr int STREAM_THREADS = THREADS + 32;     // consumer warps + the producer warp

template <typename T> struct StreamCfg;
// Tunables (overridable at build time): stages per CTA and CTAs per SM of the staged kernels.
// bf16 rows carry twice the arithmetic per byte, so they get more resident warps per SM.
#ifndef PICOSPEC_STAGES_BF16
#define PICOSPEC_STAGES_BF16 3                   // 3 x 16 KB in flight per CTA
#endif
#ifndef PICOSPEC_STAGES_F32
#define PICOSPEC_STAGES_F32 3                    // 3 x 32 KB in flight per CTA
#endif
#ifndef PICOSPEC_CTAS_PER_SM_BF16
#define PICOSPEC_CTAS_PER_SM_BF16 4              // 32 worker warps per SM at 56 registers
#endif
#ifndef PICOSPEC_CTAS_PER_SM_F32
#define PICOSPEC_CTAS_PER_SM_F32 2
#endif
#ifndef PICOSPEC_CPW_BF16
#define PICOSPEC_CPW_BF16 1                      // chunks per worker warp and tile (statistics pass)
#endif
template <> struct StreamCfg<__nv_bfloat16> {
    static constexpr int STAGES = PICOSPEC_STAGES_BF16;
    static constexpr int CTAS_PER_SM = PICOSPEC_CTAS_PER_SM_BF16;
    static constexpr int CPW = PICOSPEC_CPW_BF16;
};
template <> struct StreamCfg<float> {
    static constexpr int STAGES = PICOSPEC_STAGES_F32;
    static constexpr int CTAS_PER_SM = PICOSPEC_CTAS_PER_SM_F32;
    static constexpr int CPW = 1;
};
// tiles of the statistics pass: CPW consecutive chunks per worker warp
template <typename T> struct TileGeom {
    static constexpr int CHUNKS = TILE_CHUNKS * StreamCfg<T>::CPW;
    static constexpr int TILE_BYTES = CHUNKS * CHUNK * (int)sizeof(T);
    static constexpr int SMEM_BYTES = StreamCfg<T>::STAGES * TILE_BYTES;
};

// One chunk of a staged tile -> registers, in the lane layout of ChunkRegs (vector j of a lane is
// the 16 bytes at j*512 + lane*16 of the chunk).  v0: vocabulary index of the chunk's first entry;
// vectors at or beyond V read as -inf (V is a multiple of the vector length on this path).
__device__ __forceinline__ void load_staged(ChunkRegs<__nv_bfloat16>& r, const unsigned char* chunk, int v0, int V,
                                            int lane) {
    const uint4* p = reinterpret_cast<const uint4*>(chunk) + lane;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint4 q = p[j * 32];
        r.w[4 * j + 0] = q.x; r.w[4 * j + 1] = q.y; r.w[4 * j + 2] = q.z; r.w[4 * j + 3] = q.w;
    }
    if (v0 + CHUNK > V) {   // ragged last chunk of a row (warp-uniform)
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (v0 + j * 256 + lane * 8 >= V) r.w[4 * j + 0] = r.w[4 * j + 1] = r.w[4 * j + 2] = r.w[4 * j + 3] = 0xFF80FF80u;
    }
}
__device__ __forceinline__ void load_staged(ChunkRegs<float>& r, const unsigned char* chunk, int v0, int V, int lane) {
    const uint4* p = reinterpret_cast<const uint4*>(chunk) + lane;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint4 q = p[j * 32];
        r.f[4 * j + 0] = __uint_as_float(q.x); r.f[4 * j + 1] = __uint_as_float(q.y);
        r.f[4 * j + 2] = __uint_as_float(q.z); r.f[4 * j + 3] = __uint_as_float(q.w);
    }
    if (v0 + CHUNK > V) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (v0 + j * 128 + lane * 4 >= V) r.f[4 * j + 0] = r.f[4 * j + 1] = r.f[4 * j + 2] = r.f[4 * j + 3] = -CUDART_INF_F;
    }
}

}  // namespace picospec
