// Draft-side compression, staged variant: rows whose base, pitch and length are multiples of 16
// bytes and that hold at least one full tile.  Two kernels.
//
// compress_filter_kernel streams the rows (one CTA per row at a time, tiles of 8 chunks staged in
// shared memory by bulk async copies; the producer lane runs ahead into the next row) and keeps
// every element that can still be among the k largest:
//   - workers hold a running lower bound `thr` on the k-th largest logit of the row;
//   - per chunk a lane compares the maximum of each 16-byte vector it holds with thr; vectors
//     that reach it are parked in a per-warp ring in shared memory, and whenever 32 are parked the
//     warp tests their elements with all lanes busy and appends the survivors (64-bit keys: logit,
//     then lower index first) to the CTA's candidate buffer with one shared atomic per batch;
//   - every stored candidate is counted in a two-level histogram over the top 12 bits of the
//     orderable logit; thr is the lower edge of the highest bin whose suffix count reaches k, so
//     it is always a valid bound; it is refreshed after tiles 1, 2, 4, 8, ... and when the buffer
//     fills.  The first tile of a row gets its bound from the maxima of small groups of elements;
//   - the buffer is compacted against thr when it fills; if that is not enough an exact radix
//     select runs; a row whose candidates still do not fit (heavy ties, adversarial order) is
//     handed to the direct kernel through a redo list;
//   - with top-p the same pass accumulates the softmax normaliser relative to the first tile's
//     maximum (a row whose later logits overflow that reference also goes to the redo list).
// At the end of a row the candidates at or above thr (at least k, normally k plus a few dozen) go
// to a per-row scratch area in global memory.
//
// compress_finish_kernel (one CTA per row) sorts them and calls finish_row (top-p cut,
// renormalisation, emission, draft draw).
#pragma once
#include "compress_kernels.cuh"
#include "stream_pipeline.cuh"

namespace picospec {

constexpr int CS_CAND_CAP = 4096;    // candidate keys held in shared memory
constexpr int CS_SOFT = 2560;        // compaction trigger (leaves room for one tile's pushes)
constexpr int CS_BINS = 4096;        // histogram bins: top 12 bits of the orderable logit
constexpr int CS_SUPER = CS_BINS / 32;
constexpr int CS_QCAP = 64;          // per-warp ring of parked vectors

// row flags written by the filter kernel
constexpr int CSF_TEMPERATURE = 1, CSF_LOGIT = 2, CSF_REDO = 4, CSF_ABORT = 8;

struct CsRowMeta {
    int count;        // survivors written for the row
    int flags;
    float ref_off;    // fp32(ref * c32): reference of the streamed normaliser
    float pad;
    double z_stream;  // sum of 2^(l * c32 - ref_off) over the row (top-p only)
};

template <typename T> struct CsCfg;
template <> struct CsCfg<__nv_bfloat16> { static constexpr int STAGES = 3; };   // 3 x 16 KB
template <> struct CsCfg<float> { static constexpr int STAGES = 2; };           // 2 x 32 KB
template <typename T> struct CsGeom {
    static constexpr int TILE_BYTES = TILE_CHUNKS * CHUNK * (int)sizeof(T);
    static constexpr int STAGE_BYTES = CsCfg<T>::STAGES * TILE_BYTES;
    static constexpr int QUEUE_BYTES = WARPS * CS_QCAP * 20;
    static constexpr int SMEM_BYTES = STAGE_BYTES + CS_CAND_CAP * 8 + (CS_BINS + CS_SUPER) * 4 + QUEUE_BYTES;
};

// capacity of a row's scratch area (keys) for a sparse-row capacity k_max
__host__ __device__ __forceinline__ int cs_survivor_cap(int k_max) { return 2 * k_max > 512 ? 2 * k_max : 512; }

struct CsShared {
    float thr;          // current lower bound on the k-th largest logit
    int thr_bin;        // its bin
    unsigned top_key;   // largest orderable logit seen in the row
    int count;          // candidates appended (may run past CS_CAND_CAP: then overflow is set)
    int overflow;
    int nan;
    int abort;          // a bounded wait ran out somewhere in the CTA
    int m;              // scratch: survivor count
    double wsum[WARPS];
};

__device__ __forceinline__ int coarse_bin(float l) { return (int)(orderable(l) >> 20); }
__device__ __forceinline__ float bin_lower_edge(int bin) {
    // bins 0..7 hold -inf and the negative NaN patterns: no finite edge
    return bin <= 7 ? -CUDART_INF_F : from_orderable((uint32_t)bin << 20);
}

// ---- per-dtype pieces --------------------------------------------------------------------------

// element e of a parked vector
__device__ __forceinline__ float vec_elem(const uint4& q, int e, const __nv_bfloat16*) {
    const uint32_t w = e < 4 ? (e < 2 ? q.x : q.y) : (e < 6 ? q.z : q.w);
    return (e & 1) ? __uint_as_float(w & 0xffff0000u) : __uint_as_float(w << 16);
}
__device__ __forceinline__ float vec_elem(const uint4& q, int e, const float*) {
    return __uint_as_float(e < 2 ? (e == 0 ? q.x : q.y) : (e == 2 ? q.z : q.w));
}
__device__ __forceinline__ uint4 vec_words(const ChunkRegs<__nv_bfloat16>& r, int j) {
    return make_uint4(r.w[4 * j], r.w[4 * j + 1], r.w[4 * j + 2], r.w[4 * j + 3]);
}
__device__ __forceinline__ uint4 vec_words(const ChunkRegs<float>& r, int j) {
    return make_uint4(__float_as_uint(r.f[4 * j]), __float_as_uint(r.f[4 * j + 1]), __float_as_uint(r.f[4 * j + 2]),
                      __float_as_uint(r.f[4 * j + 3]));
}
__device__ __forceinline__ float fmax_nan(float a, float b) { return (a != a || b != b) ? CUDART_NAN_F : fmaxf(a, b); }

// Per-lane view of a chunk for the filter: which vectors may hold an element >= thr (a superset:
// the element test decides), the lane's maximum (NaN if the lane holds a NaN).
template <typename T> struct ChunkScan;
template <> struct ChunkScan<__nv_bfloat16> {
    __nv_bfloat162 vmax[4];      // per vector: (max of even elements, max of odd elements)
    float lane_max;
    __device__ __forceinline__ void scan(const ChunkRegs<__nv_bfloat16>& r) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            __nv_bfloat162 m = *reinterpret_cast<const __nv_bfloat162*>(&r.w[4 * j]);
#pragma unroll
            for (int k = 1; k < 4; ++k) m = __hmax2_nan(m, *reinterpret_cast<const __nv_bfloat162*>(&r.w[4 * j + k]));
            vmax[j] = m;
        }
        __nv_bfloat162 a = __hmax2_nan(__hmax2_nan(vmax[0], vmax[1]), __hmax2_nan(vmax[2], vmax[3]));
        const uint32_t aa = *reinterpret_cast<uint32_t*>(&a);
        const uint32_t sw = __byte_perm(aa, aa, 0x1032);
        a = __hmax2_nan(a, *reinterpret_cast<const __nv_bfloat162*>(&sw));
        lane_max = __uint_as_float(*reinterpret_cast<uint32_t*>(&a) << 16);
    }
    // thr as a packed pair: the smallest bf16 >= thr when thr is negative or a bf16 itself (every
    // threshold this kernel produces); otherwise a slightly lower value, which only adds vectors
    static __device__ __forceinline__ uint32_t pack_thr(float thr) {
        const uint32_t h = __float_as_uint(thr) >> 16;
        return h | (h << 16);
    }
    __device__ __forceinline__ bool hit(int j, uint32_t thr2) const {
        return !__hblt2(vmax[j], *reinterpret_cast<const __nv_bfloat162*>(&thr2));   // not (both halves < thr)
    }
};
template <> struct ChunkScan<float> {
    float vmax[8];
    float lane_max;
    __device__ __forceinline__ void scan(const ChunkRegs<float>& r) {
        bool nan = false;
        float lm = -CUDART_INF_F;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            vmax[j] = fmaxf(fmaxf(r.f[4 * j], r.f[4 * j + 1]), fmaxf(r.f[4 * j + 2], r.f[4 * j + 3]));
            nan |= (r.f[4 * j] != r.f[4 * j]) | (r.f[4 * j + 1] != r.f[4 * j + 1]) | (r.f[4 * j + 2] != r.f[4 * j + 2]) |
                   (r.f[4 * j + 3] != r.f[4 * j + 3]);
            lm = fmaxf(lm, vmax[j]);
        }
        lane_max = nan ? CUDART_NAN_F : lm;
    }
    static __device__ __forceinline__ uint32_t pack_thr(float thr) { return __float_as_uint(thr); }
    __device__ __forceinline__ bool hit(int j, uint32_t thr2) const { return vmax[j] >= __uint_as_float(thr2); }
};

// two-level histogram update
__device__ __forceinline__ void hist_add(unsigned* hist, int bin, unsigned v) {
    atomicAdd(&hist[bin], v);
    atomicAdd(&hist[CS_BINS + (bin >> 5)], v);
}

// Count (sign = +1) or take back (sign = -1) the maxima of groups of `g` consecutive elements of
// the lane's chunk (first tile of a row).  bf16: g in {8, 4, 2}; fp32: g in {4, 2}.
__device__ __forceinline__ void count_group_maxima(const ChunkRegs<__nv_bfloat16>& r, int g, unsigned* hist, unsigned v) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        float m4[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t w0 = r.w[4 * j + 2 * h], w1 = r.w[4 * j + 2 * h + 1];
            const float m0 = fmax_nan(__uint_as_float(w0 << 16), __uint_as_float(w0 & 0xffff0000u));
            const float m1 = fmax_nan(__uint_as_float(w1 << 16), __uint_as_float(w1 & 0xffff0000u));
            if (g == 2) {
                if (m0 == m0) hist_add(hist, coarse_bin(m0), v);
                if (m1 == m1) hist_add(hist, coarse_bin(m1), v);
            }
            m4[h] = fmax_nan(m0, m1);
            if (g == 4 && m4[h] == m4[h]) hist_add(hist, coarse_bin(m4[h]), v);
        }
        const float m8 = fmax_nan(m4[0], m4[1]);
        if (g == 8 && m8 == m8) hist_add(hist, coarse_bin(m8), v);
    }
}
__device__ __forceinline__ void count_group_maxima(const ChunkRegs<float>& r, int g, unsigned* hist, unsigned v) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float m0 = fmax_nan(r.f[4 * j], r.f[4 * j + 1]), m1 = fmax_nan(r.f[4 * j + 2], r.f[4 * j + 3]);
        if (g == 2) {
            if (m0 == m0) hist_add(hist, coarse_bin(m0), v);
            if (m1 == m1) hist_add(hist, coarse_bin(m1), v);
        } else {
            const float m = fmax_nan(m0, m1);
            if (m == m) hist_add(hist, coarse_bin(m), v);
        }
    }
}

// Warp 0: raise thr to the lower edge of the highest bin whose suffix count reaches k.
__device__ __forceinline__ void refresh_threshold(const unsigned* hist, CsShared& cs, int k, int lane) {
    // level 1: lane l owns super-bins 4l .. 4l+3 (super-bin s covers bins 32 s .. 32 s + 31)
    const uint4 sv = *reinterpret_cast<const uint4*>(&hist[CS_BINS + 4 * lane]);
    const unsigned own = sv.x + sv.y + sv.z + sv.w;
    unsigned suf = own;             // inclusive suffix sum over lanes (higher lanes = higher bins)
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned y = __shfl_down_sync(0xffffffffu, suf, d);
        if (lane + d < 32) suf += y;
    }
    const unsigned hit = __ballot_sync(0xffffffffu, suf >= (unsigned)k);
    if (!hit) return;               // fewer than k counted so far
    const int L = 31 - __clz(hit);  // highest lane whose suffix reaches k
    unsigned above = __shfl_sync(0xffffffffu, suf - own, L);      // count strictly above lane L's super-bins
    const uint4 lv = make_uint4(__shfl_sync(0xffffffffu, sv.x, L), __shfl_sync(0xffffffffu, sv.y, L),
                                __shfl_sync(0xffffffffu, sv.z, L), __shfl_sync(0xffffffffu, sv.w, L));
    int s = 4 * L + 3;
    if (above + lv.w < (unsigned)k) {
        above += lv.w;
        s = 4 * L + 2;
        if (above + lv.z < (unsigned)k) {
            above += lv.z;
            s = 4 * L + 1;
            if (above + lv.y < (unsigned)k) {
                above += lv.y;
                s = 4 * L;
            }
        }
    }
    // level 2: the 32 bins of super-bin s, lane l reads bin 32 s + l
    const unsigned h = hist[32 * s + lane];
    unsigned bs = h;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned y = __shfl_down_sync(0xffffffffu, bs, d);
        if (lane + d < 32) bs += y;
    }
    const unsigned hit2 = __ballot_sync(0xffffffffu, above + bs >= (unsigned)k);
    const int found = hit2 ? 32 * s + (31 - __clz(hit2)) : 32 * s;
    if (lane == 0 && found > cs.thr_bin) {
        cs.thr_bin = found;
        cs.thr = bin_lower_edge(found);
    }
}

// Drop the candidates below thr (all 256 workers).  Survivors go to `dst` (shared or global; may be
// `cand` itself), at most dst_cap of them are written.  Returns how many there are.
__device__ __forceinline__ int compact_candidates(const u64* cand, int n, u64* dst, int dst_cap, CsShared& cs) {
    constexpr int PER = CS_CAND_CAP / THREADS;
    const int tid = threadIdx.x;
    const uint32_t thr_key = orderable(cs.thr);
    u64 mine[PER];
#pragma unroll
    for (int e = 0; e < PER; ++e) {
        const int i = tid + e * THREADS;
        mine[e] = i < n ? cand[i] : 0ull;
    }
    if (tid == 0) cs.m = 0;
    workers_sync();
    int cnt = 0;
#pragma unroll
    for (int e = 0; e < PER; ++e) cnt += (mine[e] != 0ull && (uint32_t)(mine[e] >> 32) >= thr_key) ? 1 : 0;
    const int lane = tid & 31;
    int incl = cnt;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += y;
    }
    const int total = __shfl_sync(0xffffffffu, incl, 31);
    int base = 0;
    if (lane == 0 && total) base = atomicAdd(&cs.m, total);
    base = __shfl_sync(0xffffffffu, base, 0);
    int pos = base + incl - cnt;
#pragma unroll
    for (int e = 0; e < PER; ++e)
        if (mine[e] != 0ull && (uint32_t)(mine[e] >> 32) >= thr_key) {
            if (pos < dst_cap) dst[pos] = mine[e];
            ++pos;
        }
    workers_sync();
    return cs.m;
}

template <typename T, bool STATS>
__global__ void __launch_bounds__(STREAM_THREADS, 2) compress_filter_kernel(CompressArgs a, int tiles_per_row) {
    extern __shared__ __align__(1024) unsigned char dyn[];
    constexpr int STAGES = CsCfg<T>::STAGES;
    constexpr int TILE_BYTES = CsGeom<T>::TILE_BYTES;
    constexpr int VEC = ChunkRegs<T>::VEC, NVEC = ChunkRegs<T>::NVEC;
    constexpr bool LOGIT16 = sizeof(T) == 2;
    unsigned char* stage_mem = dyn;
    u64* cand = reinterpret_cast<u64*>(dyn + CsGeom<T>::STAGE_BYTES);
    unsigned* hist = reinterpret_cast<unsigned*>(cand + CS_CAND_CAP);          // bins, then super-bins
    unsigned char* qmem = reinterpret_cast<unsigned char*>(hist + CS_BINS + CS_SUPER);
    __shared__ __align__(8) uint64_t full[STAGES], empty[STAGES];
    __shared__ CompressShared sh;
    __shared__ CsShared cs;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rows = a.B * a.G;
    int k_eff = a.top_k > 0 ? a.top_k : a.k_max;
    if (k_eff > a.k_max) k_eff = a.k_max;
    if (k_eff > a.V) k_eff = a.V;
    const int surv_cap = cs_survivor_cap(a.k_max);

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], WARPS);
        }
        mbar_init_fence();
        if (blockIdx.x == 0) {
            *a.queue_count_next = 0;
            *a.redo_count_next = 0;
        }
        cs.thr = -CUDART_INF_F;
        cs.thr_bin = 0;
        cs.top_key = 0u;
        cs.count = 0;
        cs.overflow = 0;
        cs.nan = 0;
        cs.abort = 0;
    }
    for (int i = tid; i < CS_BINS + CS_SUPER; i += STREAM_THREADS) hist[i] = 0u;
    __syncthreads();

    if (warp == WARPS) {
        // ---- producer: every tile of every row of this CTA, in order -------------------------
        if (lane != 0) return;
        const uint64_t pol = l2_evict_first_policy();
        uint32_t i = 0;
        for (int row = blockIdx.x; row < rows; row += gridDim.x) {
            const bool valid = temp_ok(a.temperature[row / a.G]);
            const T* rowp = reinterpret_cast<const T*>(a.logits) + (long long)row * a.row_stride;
            for (int ti = 0; ti < tiles_per_row; ++ti, ++i) {
                const int s = (int)(i % STAGES);
                const uint32_t round = i / STAGES;
                if (round > 0 && !mbar_wait(&empty[s], (round - 1) & 1)) {
                    atomicOr(a.status, ST_INTERNAL);
                    return;
                }
                if (valid) {
                    const int v0 = ti * TILE_CHUNKS * CHUNK;
                    const int v1 = min(a.V, v0 + TILE_CHUNKS * CHUNK);
                    const uint32_t bytes = (uint32_t)(v1 - v0) * (uint32_t)sizeof(T);
                    mbar_arrive_expect_tx(&full[s], bytes);
                    bulk_load(stage_mem + s * TILE_BYTES, rowp + v0, bytes, &full[s], pol);
                } else {
                    mbar_arrive(&full[s]);
                }
            }
        }
        return;
    }

    // ---- workers ------------------------------------------------------------------------------
    uint4* qvec = reinterpret_cast<uint4*>(qmem) + warp * CS_QCAP;
    int* qidx = reinterpret_cast<int*>(qmem + WARPS * CS_QCAP * 16) + warp * CS_QCAP;
    const unsigned lt_mask = (1u << lane) - 1u;
    // group size of the first-tile bound: at least 4 k groups in the tile
    int g = VEC;
    while (g > 2 && (TILE_CHUNKS * CHUNK) / g < 4 * k_eff) g >>= 1;

    bool dead = false;      // this warp stopped waiting on copies; it still joins every barrier
    uint32_t i = 0;
    for (int row = blockIdx.x; row < rows; row += gridDim.x) {
        const int b = row / a.G;
        const float Tb = a.temperature[b];
        const bool valid = temp_ok(Tb);
        const float c32 = temp_scale(Tb);
        float ref_off = 0.f, acc = 0.f;
        int qhead = 0, qn = 0;
        bool skip = false;   // row overflowed: consume its tiles without work

        // tests up to 32 parked vectors with all lanes busy and appends the survivors
        auto drain = [&](int n) {
            const bool active = lane < n;
            const int slot = (qhead + lane) & (CS_QCAP - 1);
            uint4 q = make_uint4(0, 0, 0, 0);
            int vb = a.V;
            if (active) {
                q = qvec[slot];
                vb = qidx[slot];
            }
            const float thr = *(volatile float*)&cs.thr;
            unsigned pass = 0;
            if (vb < a.V) {
#pragma unroll
                for (int e = 0; e < VEC; ++e)
                    if (vec_elem(q, e, (const T*)nullptr) >= thr) pass |= 1u << e;
            }
            const int cnt = __popc(pass);
            int incl = cnt;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += y;
            }
            const int total = __shfl_sync(0xffffffffu, incl, 31);
            if (total) {
                int base = 0;
                if (lane == 0) base = atomicAdd(&cs.count, total);
                base = __shfl_sync(0xffffffffu, base, 0);
                int pos = base + incl - cnt;
                while (pass) {
                    const int e = __ffs(pass) - 1;
                    pass &= pass - 1;
                    if (pos < CS_CAND_CAP) {
                        const float l = vec_elem(q, e, (const T*)nullptr);
                        cand[pos] = make_key(l, vb + e);
                        hist_add(hist, coarse_bin(l), 1u);
                    } else {
                        cs.overflow = 1;
                    }
                    ++pos;
                }
            }
            qhead = (qhead + n) & (CS_QCAP - 1);
            qn -= n;
            __syncwarp();       // the slots just read may be refilled
        };

        for (int ti = 0; ti < tiles_per_row; ++ti, ++i) {
            const int s = (int)(i % STAGES);
            const uint32_t round = i / STAGES;
            if (!dead && !mbar_wait(&full[s], round & 1)) {
                dead = true;
                if (lane == 0) {
                    cs.abort = 1;
                    atomicOr(a.status, ST_INTERNAL);
                }
            }
            const int c = ti * TILE_CHUNKS + warp;
            const bool work = !dead && valid && !skip && c < a.nch;
            ChunkRegs<T> regs;
            if (work) load_staged(regs, stage_mem + s * TILE_BYTES + warp * (CHUNK * (int)sizeof(T)), c * CHUNK, a.V, lane);
            __syncwarp();
            if (lane == 0 && !dead) mbar_arrive(&empty[s]);

            ChunkScan<T> sc;
            if (work) {
                sc.scan(regs);
                if (sc.lane_max != sc.lane_max) cs.nan = 1;
            }
            if (ti == 0 && valid) {
                // first tile (every warp holds a full chunk): bound from the maxima of groups of g
                // elements, counted in the histogram for the scan and taken back afterwards
                if (work) {
                    count_group_maxima(regs, g, hist, 1u);
                    const float wm = warp_max(sc.lane_max);      // NaN lanes are ignored here
                    if (lane == 0 && wm == wm) atomicMax(&cs.top_key, orderable(wm));
                }
                workers_sync();
                if (warp == 0) refresh_threshold(hist, cs, k_eff, lane);
                if (STATS) ref_off = __fmul_rn(from_orderable(*(volatile unsigned*)&cs.top_key), c32);
                workers_sync();
                if (work) count_group_maxima(regs, g, hist, 0xffffffffu);
            } else if (work) {
                const unsigned lk = orderable(sc.lane_max);      // NaN maps above every number: harmless
                if (sc.lane_max == sc.lane_max && lk > *(volatile unsigned*)&cs.top_key) atomicMax(&cs.top_key, lk);
            }
            if (work) {
                if (STATS) acc += lane_exp_sum2(regs, c32, ref_off);
                const uint32_t thr2 = ChunkScan<T>::pack_thr(*(volatile float*)&cs.thr);
                const int v0 = c * CHUNK;
#pragma unroll
                for (int j = 0; j < NVEC; ++j) {
                    const bool hit = sc.hit(j, thr2);
                    const unsigned m = __ballot_sync(0xffffffffu, hit);
                    if (m) {
                        if (hit) {
                            const int slot = (qhead + qn + __popc(m & lt_mask)) & (CS_QCAP - 1);
                            qvec[slot] = vec_words(regs, j);
                            qidx[slot] = v0 + j * (32 * VEC) + lane * VEC;
                        }
                        qn += __popc(m);
                        __syncwarp();
                        if (qn >= 32) drain(32);
                    }
                }
            }
            const bool last = ti + 1 == tiles_per_row;
            const bool refresh_due = last || ((ti + 1) & ti) == 0;     // after tiles 1, 2, 4, 8, ...
            if (refresh_due && qn > 0) drain(qn);      // the histogram must be complete for a refresh

            // ---- tile boundary ----------------------------------------------------------------
            // One barrier that also ORs every warp's view of "the buffer needs attention".  The
            // counters only grow while warps push, and the last warp to arrive sees their final
            // values, so the OR is the same decision for everybody.
            const bool attention = workers_sync_or(*(volatile int*)&cs.count > CS_SOFT ||
                                                   *(volatile int*)&cs.overflow != 0 ||
                                                   *(volatile int*)&cs.abort != 0);
            if (attention) {
                if (qn > 0) drain(qn);
                workers_sync();                     // all pushes are in
                int n = *(volatile int*)&cs.count;
                const bool ovf = *(volatile int*)&cs.overflow != 0;
                if (*(volatile int*)&cs.abort) dead = true;
                workers_sync();                     // everybody has read the counters
                if (valid && !skip) {
                    if (ovf) {
                        skip = true;
                    } else {
                        if (warp == 0) refresh_threshold(hist, cs, k_eff, lane);
                        workers_sync();
                        if (n > CS_SOFT && !last) {
                            n = compact_candidates(cand, n, cand, CS_CAND_CAP, cs);
                            if (n > CS_SOFT) {
                                // ties or a coarse bin too full: exact selection of the k best so far
                                const u64 kth = keep_top_k<LOGIT16>(cand, reinterpret_cast<u64*>(qmem), n, k_eff, sh);
                                n = k_eff;
                                if (tid == 0) {
                                    const float tl = key_logit(kth);
                                    if (tl > cs.thr) {
                                        cs.thr = tl;
                                        cs.thr_bin = coarse_bin(tl);
                                    }
                                }
                            }
                            if (tid == 0) cs.count = n;
                            workers_sync();
                        }
                    }
                }
            } else if (refresh_due && valid && !skip) {
                if (warp == 0) refresh_threshold(hist, cs, k_eff, lane);
                workers_sync();
            }
        }

        // ---- row end: survivors and row statistics to global scratch -----------------------------
        if (STATS) {
            const double sw = (double)warp_sum(acc);
            if (lane == 0) cs.wsum[warp] = sw;
        }
        workers_sync();
        int flags = 0;
        int m = 0;
        if (dead || *(volatile int*)&cs.abort) {
            flags = CSF_ABORT;
        } else if (!valid) {
            flags = CSF_TEMPERATURE;
        } else if (skip || *(volatile int*)&cs.overflow) {
            flags = CSF_REDO;
        } else {
            u64* dst = a.surv_keys + (long long)row * surv_cap;
            const int n = cs.count;
            m = compact_candidates(cand, n, dst, surv_cap, cs);
            if (m > surv_cap) {
                // too many ties at the bound for the scratch area: exact selection here
                m = compact_candidates(cand, n, cand, CS_CAND_CAP, cs);
                keep_top_k<LOGIT16>(cand, reinterpret_cast<u64*>(qmem), m, k_eff, sh);
                for (int x = tid; x < k_eff; x += THREADS) dst[x] = cand[x];
                m = k_eff;
            }
            if (cs.nan || m < k_eff) flags = CSF_LOGIT;
        }
        if (tid == 0) {
            double zs = 0.0;
            if (STATS)
                for (int w = 0; w < WARPS; ++w) zs += cs.wsum[w];
            // a reference that later logits overflowed, or NaN / +inf data: the direct kernel sorts it out
            if (STATS && flags == 0 && !(zs > 0.0 && zs < CUDART_INF)) flags = CSF_REDO;
            if (flags & CSF_REDO) a.redo_rows[atomicAdd(a.redo_count, 1)] = row;
            CsRowMeta meta;
            meta.count = m;
            meta.flags = flags;
            meta.ref_off = ref_off;
            meta.pad = 0.f;
            meta.z_stream = zs;
            a.surv_meta[row] = meta;
        }
        workers_sync();
        // reset the row state
        for (int x = tid; x < CS_BINS + CS_SUPER; x += THREADS) hist[x] = 0u;
        if (tid == 0) {
            cs.thr = -CUDART_INF_F;
            cs.thr_bin = 0;
            cs.top_key = 0u;
            cs.count = 0;
            cs.overflow = 0;
            cs.nan = 0;
        }
        workers_sync();
    }
}

// One CTA per row: sort the survivors, then cut / renormalise / emit.
template <typename T, bool STATS>
__global__ void __launch_bounds__(THREADS) compress_finish_kernel(CompressArgs a) {
    extern __shared__ u64 keys[];          // [pow2 >= survivors]
    __shared__ CompressShared sh;
    const int tid = threadIdx.x;
    const int row = blockIdx.x;
    int k_eff = a.top_k > 0 ? a.top_k : a.k_max;
    if (k_eff > a.k_max) k_eff = a.k_max;
    if (k_eff > a.V) k_eff = a.V;
    const CsRowMeta meta = a.surv_meta[row];
    if (meta.flags & CSF_REDO) return;                 // the direct kernel writes this row
    if (meta.flags) {
        emit_invalid_row(a, row);
        if (tid == 0 && (meta.flags & (CSF_TEMPERATURE | CSF_LOGIT)))
            atomicOr(a.status, (meta.flags & CSF_TEMPERATURE) ? ST_TEMPERATURE : ST_LOGIT);
        return;
    }
    const int m = meta.count;
    int n2 = 1;
    while (n2 < m) n2 <<= 1;
    const u64* src = a.surv_keys + (long long)row * cs_survivor_cap(a.k_max);
    for (int x = tid; x < n2; x += THREADS) keys[x] = x < m ? src[x] : 0ull;
    bitonic_sort_desc(keys, n2);
    const float top = key_logit(keys[0]);
    const float Tb = a.temperature[row / a.G];
    double Z = 0.0;
    if (STATS) {
        // move the streamed sum from its reference onto the scale of the weights exp(l/T - top/T)
        const float c32 = temp_scale(Tb);
        Z = meta.z_stream * exp2((double)meta.ref_off - (double)top * (double)c32);
    }
    const bool bad = !(top > -CUDART_INF_F) || !(top < CUDART_INF_F) || (STATS && !(Z > 0.0));
    if (bad) {
        emit_invalid_row(a, row);
        if (tid == 0) atomicOr(a.status, ST_LOGIT);
        return;
    }
    finish_row<false>(a, row, keys, k_eff, Tb, Z, sh);
}

}  // namespace picospec
