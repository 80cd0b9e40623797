// Draft-side compression, staged variant: rows whose base, pitch and length are multiples of 16
// bytes and that hold at least one full tile.  Two kernels.
//
// compress_filter_kernel streams the rows (one CTA per row at a time, tiles of 8 chunks staged in
// shared memory by bulk async copies; the producer lane runs ahead into the next row) and keeps
// every element that can still be among the k largest:
//   - the CTA holds a running lower bound `thr` on the k-th largest logit of the row;
//   - per chunk a lane compares its 32 values with thr (packed compares for bf16) into a 32-bit
//     mask; the warp then takes one set bit per lane per step, ranks the lanes by ballot and
//     appends the values (64-bit keys: logit, then lower index first; the value is re-read from the
//     staged tile) to the warp's own region of the candidate buffer: no atomics with a return
//     value, no CTA barrier.  About 15 of the 1024 values of a chunk pass, so this is two or three
//     steps per chunk;
//   - every stored candidate is counted in a two-level histogram whose bins count up from the
//     first tile's bound, one bin per 16-bit logit code (the top 16 bits of the orderable key: a
//     bf16 value, 2^-7 relative for fp32), magnitudes below 2^-10 sharing one bin on each side of
//     zero so that a window that crosses zero does not spend itself on tiny exponents; 4096 bins
//     reach 32 binades up, whatever lies beyond shares the last bin; thr is the lower edge of the
//     highest bin whose suffix count reaches k, so it is a valid bound whenever it is computed,
//     by any warp, from whatever has been counted so far.
//     The warps take turns refreshing it, once per tile; a warp whose region fills refreshes it
//     and drops its candidates below it;
//   - the first tile of a row gets its bound without the histogram: every warp finds, by a
//     16-step bisection over its own chunk, a value that at least ceil(k/8) of its small groups
//     of elements reach with their maximum; the smallest of the eight values is reached by at
//     least k elements of the tile (one CTA barrier, the only one inside a row);
//   - a row whose candidates do not fit (heavy ties, adversarial order) is handed to the direct
//     kernel through a redo list;
//   - with top-p the same pass accumulates the softmax normaliser relative to the first tile's
//     maximum (a row whose later logits overflow that reference also goes to the redo list).
// At the end of a row the candidates at or above thr (at least k; for 16-bit logits the k best plus
// the ties of the k-th, for 32-bit logits plus what shares its 16-bit code) go to a per-row scratch
// area in global memory, with the bound itself.
//
// compress_finish_kernel (one CTA per row) trims them to k where that is cheap, sorts them with a
// bitonic network held in registers and calls finish_row (top-p cut, renormalisation, emission,
// draft draw).
#pragma once
#include "compress_kernels.cuh"


#include "stream_pipeline.cuh"

namespace picospec {

// Two shapes of the filter kernel, both sized for three CTAs per SM on 16-bit rows (the kernel is
// bound by instruction issue, so resident warps count for more than tiles in flight: two stages
// measure the same as three, three CTAs 15 % faster than two).  Rows with k <= 512 need few live
// candidates: a small candidate buffer and three stages of 16 KB; larger k takes the big buffer and
// two stages.  32-bit rows have 32 KB tiles: two stages and two CTAs per SM in both shapes.
constexpr int CS_CAP_SMALL = 2048, CS_CAP_LARGE = 4096;    // candidate keys held in shared memory
constexpr int CS_K_SMALL = 512;                            // largest k served by the small shape
constexpr int CS_BINS = 4096;        // histogram bins above the first tile's bound; the last one is open-ended
constexpr int CS_DEAD = 117 << 7;    // 16-bit magnitude codes below 2^-10: one bin on each side of zero
constexpr int CS_SUPER = CS_BINS / 32;
// Bin counts are 16 bits wide, two per word (super-bin counts are 32-bit).  A count can only wrap
// on rows that push tens of thousands of values into one bin; a wrap makes a sum too small (a
// lower, still valid bound) and its carry makes the neighbouring bin one too large, which can at
// worst leave fewer than k survivors: such a row goes to the redo list.
constexpr int CS_HIST_WORDS = CS_BINS / 2 + CS_SUPER;

// row flags written by the filter kernel
constexpr int CSF_TEMPERATURE = 1, CSF_LOGIT = 2, CSF_REDO = 4, CSF_ABORT = 8, CSF_RANGE = 16;

struct CsRowMeta {
    int count;        // survivors written for the row
    int flags;
    float ref_off;    // fp32(ref * c32): reference of the streamed normaliser
    unsigned thr_key; // the row's final bound: every survivor's orderable logit is at least this
    double z_stream;  // sum of 2^(l * c32 - ref_off) over the row (top-p only)
};

// bf16 SMALL: CAP 2048, 3 stages x 16 KB; bf16 LARGE: CAP 4096, 2 stages x 16 KB (72.5 KB either way:
// 3 CTAs / SM).  fp32: 2 stages x 32 KB (88.5 / 104.5 KB: 2 CTAs / SM).
template <typename T, bool SMALL> struct CsGeom {
    static constexpr int CAP = SMALL ? CS_CAP_SMALL : CS_CAP_LARGE;
    static constexpr int REGION = CAP / WARPS;             // each worker warp appends to its own region
    static constexpr int STAGES = (sizeof(T) == 2 && SMALL) ? 3 : 2;
    static constexpr int CTAS = sizeof(T) == 2 ? 3 : 2;
    static constexpr int TILE_BYTES = TILE_CHUNKS * CHUNK * (int)sizeof(T);
    static constexpr int STAGE_BYTES = STAGES * TILE_BYTES;
    static constexpr int SMEM_BYTES = STAGE_BYTES + CAP * 8 + CS_HIST_WORDS * 4;
};

// capacity of a row's scratch area (keys) for a sparse-row capacity k_max
__host__ __device__ __forceinline__ int cs_survivor_cap(int k_max) { return 2 * k_max > 512 ? 2 * k_max : 512; }

struct CsShared {
    unsigned thr_key;   // orderable form of the current lower bound on the k-th largest logit
    unsigned thr0_key;  // first-tile bound: minimum over the warps' own bounds
    unsigned top_key;   // largest orderable logit of the first tile
    int overflow;       // a region ran out of room: the row goes to the redo list
    int nan;
    int m;              // survivors written at the end of the piece
    double wsum[WARPS];
};
// state of the CTA that outlives a piece
struct CsCta {
    int abort;          // a bounded wait ran out somewhere in the CTA
    int wcnt[WARPS];    // per warp: entries in its region (the slot counter its lanes draw from)
};
__device__ __forceinline__ void cs_reset(CsShared& cs) {
    cs.thr_key = 0u;
    cs.thr0_key = 0xffffffffu;
    cs.top_key = 0u;
    cs.overflow = 0;
    cs.nan = 0;
    cs.m = 0;
}

// threshold (a float) of an orderable key; keys below 0x00800000 are -inf and the negative NaN patterns
__device__ __forceinline__ float thr_of_key(unsigned key) {
    return key < 0x00800000u ? -CUDART_INF_F : from_orderable(key);
}

// ---- per-dtype pieces --------------------------------------------------------------------------

// 32-bit mask of the lane's values that are >= thr (NaN never passes).
//   bf16: bit k = low half of word k, bit 16 + k = high half of word k.  The packed threshold is
//         the smallest bf16 >= thr for every threshold this kernel produces (a bf16 value itself,
//         or the lower edge of a histogram bin: positive edges are bf16 values, negative edges
//         have all low bits set, so dropping them rounds towards zero, i.e. up).
//   fp32: bit k = value k.
__device__ __forceinline__ unsigned pass_mask(const ChunkRegs<__nv_bfloat16>& r, float thr) {
    const uint32_t h = __float_as_uint(thr) >> 16;
    const uint32_t t2 = h | (h << 16);
    const __nv_bfloat162 t = *reinterpret_cast<const __nv_bfloat162*>(&t2);
    unsigned mask = 0;
#pragma unroll
    for (int k = 0; k < 16; ++k)
        mask |= __hge2_mask(*reinterpret_cast<const __nv_bfloat162*>(&r.w[k]), t) & (0x00010001u << k);
    return mask;
}
__device__ __forceinline__ unsigned pass_mask(const ChunkRegs<float>& r, float thr) {
    unsigned mask = 0;
#pragma unroll
    for (int k = 0; k < 32; ++k) mask |= (r.f[k] >= thr ? 1u : 0u) << k;
    return mask;
}
// offset inside the chunk (in elements) of the value behind mask bit b of a lane
__device__ __forceinline__ int bit_offset(int b, int lane, const __nv_bfloat16*) {
    const int k = b & 15;
    return (k >> 2) * 256 + lane * 8 + (k & 3) * 2 + (b >> 4);
}
__device__ __forceinline__ int bit_offset(int b, int lane, const float*) { return (b >> 2) * 128 + lane * 4 + (b & 3); }
// value at an element offset of a staged chunk
__device__ __forceinline__ float staged_value(const unsigned char* chunk, int off, const __nv_bfloat16*) {
    return __uint_as_float((uint32_t)reinterpret_cast<const unsigned short*>(chunk)[off] << 16);
}
__device__ __forceinline__ float staged_value(const unsigned char* chunk, int off, const float*) {
    return reinterpret_cast<const float*>(chunk)[off];
}

// 16-bit orderable keys of the maxima of groups of 2 consecutive elements of the lane's chunk
// (NaN is ignored here).
__device__ __forceinline__ void pair_keys(const ChunkRegs<__nv_bfloat16>& r, unsigned (&key)[16]) {
#pragma unroll
    for (int k = 0; k < 16; ++k)
        key[k] = orderable(fmaxf(__uint_as_float(r.w[k] << 16), __uint_as_float(r.w[k] & 0xffff0000u))) >> 16;
}
__device__ __forceinline__ void pair_keys(const ChunkRegs<float>& r, unsigned (&key)[16]) {
#pragma unroll
    for (int k = 0; k < 16; ++k) key[k] = orderable(fmaxf(r.f[2 * k], r.f[2 * k + 1])) >> 16;
}

// Warp-wide search, two bits per step: the largest 16-bit key t such that at least `need` of the
// warp's G*32 group keys are >= t (the need-th largest key).  G in {4, 8, 16} keys per lane.
template <int G>
__device__ __forceinline__ unsigned warp_kth_key(const unsigned (&key)[16], int need) {
    unsigned prefix = 0;
#pragma unroll 1
    for (int bit = 14; bit >= 0; bit -= 2) {
        const unsigned t1 = prefix | (1u << bit), t2 = prefix | (2u << bit), t3 = prefix | (3u << bit);
        int c1 = 0, c2 = 0, c3 = 0;
#pragma unroll
        for (int x = 0; x < G; ++x) {
            c1 += key[x] >= t1 ? 1 : 0;
            c2 += key[x] >= t2 ? 1 : 0;
            c3 += key[x] >= t3 ? 1 : 0;
        }
        c1 = __reduce_add_sync(0xffffffffu, c1);
        c2 = __reduce_add_sync(0xffffffffu, c2);
        c3 = __reduce_add_sync(0xffffffffu, c3);
        prefix = c3 >= need ? t3 : c2 >= need ? t2 : c1 >= need ? t1 : prefix;
    }
    return prefix;
}

// First-tile bound of one warp: group size g (elements) in {2, 4, 8 (bf16 only)}.  (Inlined: an
// out-of-line call would force the chunk registers through local memory in every tile.)
template <typename T>
__device__ __forceinline__ unsigned first_tile_key(const ChunkRegs<T>& regs, int g, int need) {
    unsigned key[16];
    if (g == ChunkRegs<T>::VEC) {
        // groups = the lane's 16-byte vectors: their maxima come packed
        constexpr int NV = ChunkRegs<T>::NVEC;
#pragma unroll
        for (int j = 0; j < NV; ++j) key[j] = orderable(regs.vec_max(j)) >> 16;
        return warp_kth_key<NV>(key, need);
    }
    pair_keys(regs, key);
    if (g == 2) return warp_kth_key<16>(key, need);
#pragma unroll
    for (int x = 0; x < 8; ++x) key[x] = max(key[2 * x], key[2 * x + 1]);
    if (g == 4) return warp_kth_key<8>(key, need);
#pragma unroll
    for (int x = 0; x < 4; ++x) key[x] = max(key[2 * x], key[2 * x + 1]);
    return warp_kth_key<4>(key, need);
}

// two-level histogram update
// Bin coordinate of a 16-bit orderable code (monotone): the code itself with the magnitudes
// below 2^-10 squeezed onto 0x7FFF (negative side) and 0x8000 (positive side).
__device__ __forceinline__ int bin_coord(unsigned o16) {
    const bool pos = o16 >= 0x8000u;
    const int mag = pos ? (int)o16 - 0x8000 : 0x7FFF - (int)o16;
    const int c = max(mag - CS_DEAD, 0);
    return pos ? 0x8000 + c : 0x7FFF - c;
}
// smallest 16-bit code whose coordinate is at least G
__device__ __forceinline__ unsigned coord_code(int G) {
    if (G >= 0x8000) {
        const int c = G - 0x8000;
        return (unsigned)(c ? 0x8000 + c + CS_DEAD : 0x8000);
    }
    return (unsigned)(0x7FFF - ((0x7FFF - G) + CS_DEAD));
}
// bin of an orderable key at or above the first tile's bound (coordinate g0)
__device__ __forceinline__ int hist_bin(unsigned okey, int g0) {
    return min(bin_coord(okey >> 16) - g0, CS_BINS - 1);
}
__device__ __forceinline__ void hist_add(unsigned* hist, int bin) {
    atomicAdd(&hist[bin >> 1], (bin & 1) ? 0x10000u : 1u);
    atomicAdd(&hist[CS_BINS / 2 + (bin >> 5)], 1u);
}

// One warp: the highest bin whose suffix count (itself and every bin above it) reaches k, or -1 if
// fewer than k values have been counted.
__device__ __forceinline__ int kth_bin(const unsigned* hist, int k, int lane) {
    // level 1: lane l owns super-bins 4l .. 4l+3 (super-bin s covers bins 32 s .. 32 s + 31)
    const uint4 sv = *reinterpret_cast<const uint4*>(&hist[CS_BINS / 2 + 4 * lane]);
    const unsigned own = sv.x + sv.y + sv.z + sv.w;
    unsigned suf = own;             // inclusive suffix sum over lanes (higher lanes = higher bins)
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned y = __shfl_down_sync(0xffffffffu, suf, d);
        if (lane + d < 32) suf += y;
    }
    const unsigned hit = __ballot_sync(0xffffffffu, suf >= (unsigned)k);
    if (!hit) return -1;            // fewer than k counted so far
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
    unsigned bs = (hist[16 * s + (lane >> 1)] >> ((lane & 1) * 16)) & 0xffffu;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned y = __shfl_down_sync(0xffffffffu, bs, d);
        if (lane + d < 32) bs += y;
    }
    const unsigned hit2 = __ballot_sync(0xffffffffu, above + bs >= (unsigned)k);
    return hit2 ? 32 * s + (31 - __clz(hit2)) : 32 * s;
}

// One warp: raise thr to the lower edge of the highest bin whose suffix count reaches k.
__device__ __forceinline__ void refresh_threshold(const unsigned* hist, CsShared& cs, int k, int lane) {
    const int found = kth_bin(hist, k, lane);
    if (found >= 0 && lane == 0) {
        const int g0 = bin_coord(*(volatile unsigned*)&cs.thr0_key >> 16);
        atomicMax(&cs.thr_key, coord_code(g0 + found) << 16);
    }
}

// Warp-local: drop the entries of this warp's region below thr (stable, in place).
__device__ __forceinline__ int compact_region(u64* region, int n, unsigned thr_key, int lane) {
    int out = 0;
    for (int base = 0; base < n; base += 32) {
        const int i = base + lane;
        const u64 key = i < n ? region[i] : 0ull;
        const bool keep = i < n && (unsigned)(key >> 32) >= thr_key;
        const unsigned m = __ballot_sync(0xffffffffu, keep);
        if (keep) region[out + __popc(m & ((1u << lane) - 1u))] = key;
        out += __popc(m);
    }
    __syncwarp();
    return out;
}

// Refresh the bound (one warp; out of line).
__device__ __noinline__ void refresh_bound(int hist_off, CsShared* cs, int k_eff) {
    extern __shared__ __align__(1024) unsigned char dyn[];
    refresh_threshold(reinterpret_cast<const unsigned*>(dyn + hist_off), *cs, k_eff, threadIdx.x & 31);
}
// Region nearly full: bring the bound up to date and drop what fell below it (one warp; out of line).
// The warp's slot counter follows.
__device__ __noinline__ int maintain_region(int wcount, int region_off, int hist_off, CsShared* cs, int* wcnt, int k_eff) {
    extern __shared__ __align__(1024) unsigned char dyn[];
    const int lane = threadIdx.x & 31;
    refresh_threshold(reinterpret_cast<const unsigned*>(dyn + hist_off), *cs, k_eff, lane);
    __syncwarp();
    const int n = compact_region(reinterpret_cast<u64*>(dyn + region_off), wcount, *(volatile unsigned*)&cs->thr_key, lane);
    if (lane == 0) *wcnt = n;
    __syncwarp();
    return n;
}

// ---- how the rows of a call are dealt to the CTAs of the filter kernel ----------------------------
// With rows = q * grid + rem, CTA b first takes the q whole rows b, b + grid, ... (so that at any time
// the CTAs read one window of memory that moves forward, as a copy would).  The rem rows that
// are left would keep only some of the CTAs busy for a whole row's time, so each of them is cut into
// `split` pieces of consecutive tiles and the rem * split pieces are dealt round-robin: piece n goes
// to CTA n % grid.  A piece is filtered on its own: it keeps a bound that at least k of ITS elements
// reach, which is a valid bound for the row, and leaves its survivors in its own scratch area (whole
// row r: area r; tail piece n: area rows + n).  The finish kernel puts the pieces of a row together.
// No piece starts at a row's last tile when that tile is ragged (the first tile of a piece must be a
// full one).
struct FilterPlan {
    int tiles_per_row;
    int ragged_last;        // the last tile of a row holds fewer than TILE_CHUNKS full chunks
    int grid;               // CTAs of the filter kernel
    int rows;
    int q;                  // whole rows per CTA
    int rem;                // rows dealt in pieces: rows q * grid .. rows - 1
    int split;              // pieces per such row
};
// first tile of piece p (0 .. split) of a split row
__host__ __device__ __forceinline__ int plan_piece_tile(const FilterPlan& p, int piece) {
    int c = p.tiles_per_row * piece / p.split;
    if (p.ragged_last && p.tiles_per_row > 1 && c < p.tiles_per_row && c == p.tiles_per_row - 1) --c;
    return c;
}
// The k-th unit of work of CTA b: a whole row or a piece of a tail row.  false: no more work.
struct FilterPiece {
    int row, tile0, tile1, area;
};
__host__ __device__ __forceinline__ bool plan_piece(const FilterPlan& p, int b, int k, FilterPiece& out) {
    if (k < p.q) {
        out.row = k * p.grid + b;      // the CTAs advance through memory side by side
        out.tile0 = 0;
        out.tile1 = p.tiles_per_row;
        out.area = out.row;
        return true;
    }
    const long long n = (long long)b + (long long)(k - p.q) * p.grid;
    if (n >= (long long)p.rem * p.split) return false;
    const int j = (int)(n / p.split), pc = (int)(n - (long long)j * p.split);
    out.row = p.q * p.grid + j;
    out.tile0 = plan_piece_tile(p, pc);
    out.tile1 = plan_piece_tile(p, pc + 1);
    out.area = p.rows + (int)n;
    return true;        // (tile0 == tile1: an empty piece, skipped by everyone)
}
// Host side: the plan for `rows` rows on `slots` resident CTAs.  Rows are cut only when a CTA gets at most
// one whole row (few rows per CTA: the remainder decides the kernel's length); the split is then the one
// that shortens the tail most among those that keep a piece at least two tiles long and the number of
// pieces within 2 * grid (the scratch areas are sized for that).
inline FilterPlan make_filter_plan(int rows, int tiles_per_row, bool ragged_last, long long slots) {
    FilterPlan p;
    p.tiles_per_row = tiles_per_row;
    p.ragged_last = ragged_last ? 1 : 0;
    p.rows = rows;
    long long g = slots < 1 ? 1 : slots;
    const long long most = (long long)rows * (tiles_per_row >= 2 ? tiles_per_row / 2 : 1);   // pieces of two tiles
    if (g > most) g = most;
    if (g < 1) g = 1;
    p.grid = (int)g;
    p.q = (int)(rows / g);
    p.rem = (int)(rows - (long long)p.q * g);
    p.split = 1;
    // Pieces pay the per-piece work (first-tile bound, hand-over) again; that is worth it only while
    // the remainder is a large part of what a CTA does.
    if (p.rem > 0 && p.q <= 1) {
        double best = 1e9;
        const int smax = tiles_per_row >= 2 ? tiles_per_row / 2 : 1;
        for (int sp = 1; sp <= 8 && sp <= smax && (long long)p.rem * sp <= 2 * g; ++sp) {
            const long long per_cta = ((long long)p.rem * sp + g - 1) / g;      // pieces the busiest CTA gets
            const double cost = (double)per_cta / sp;
            if (cost < best - 1e-9) {
                best = cost;
                p.split = sp;
            }
        }
    }
    return p;
}

// First-tile bound of one warp when it needs at most 32 elements (k <= 256): the lanes form at
// least `need` groups of `group_lanes` lanes (a power of two); every group's largest value is
// reached by one element of the group, so the smallest of the group maxima is reached by at least
// `need` elements of the warp's chunk.  Returns its 16-bit orderable code (rounded down).
__device__ __forceinline__ unsigned first_tile_key_groups(float lane_max, int group_lanes) {
    unsigned key = orderable(lane_max) >> 16;
    for (int d = 1; d < group_lanes; d <<= 1) key = max(key, __shfl_xor_sync(0xffffffffu, key, d));
    return __reduce_min_sync(0xffffffffu, key);
}

template <typename T, bool STATS, bool SMALL>
__global__ void __launch_bounds__(STREAM_THREADS, CsGeom<T, SMALL>::CTAS)
compress_filter_kernel(CompressArgs a, FilterPlan plan, unsigned long long wait_limit_ns) {
    extern __shared__ __align__(1024) unsigned char dyn[];
    typedef CsGeom<T, SMALL> Geom;
    constexpr int STAGES = Geom::STAGES;
    constexpr int TILE_BYTES = Geom::TILE_BYTES;
    constexpr int CS_CAND_CAP = Geom::CAP, CS_REGION = Geom::REGION;
    constexpr int VEC = ChunkRegs<T>::VEC;
    unsigned char* stage_mem = dyn;
    u64* cand = reinterpret_cast<u64*>(dyn + Geom::STAGE_BYTES);
    unsigned* hist = reinterpret_cast<unsigned*>(cand + CS_CAND_CAP);          // bins, then super-bins
    __shared__ __align__(8) uint64_t full[STAGES], empty[STAGES];
    // Two copies of the per-piece state, used in turn: the copy of the piece that has just ended is
    // reset by one thread while the other warps already start on the next piece.
    __shared__ CsShared css[2];
    __shared__ CsCta cta;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
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
        cs_reset(css[0]);
        cs_reset(css[1]);
        cta.abort = 0;
    }
    if (tid < WARPS) cta.wcnt[tid] = 0;
    for (int i = tid; i < CS_HIST_WORDS; i += STREAM_THREADS) hist[i] = 0u;
    grid_dependency_sync();
    if (tid == 0 && blockIdx.x == 0) {
        *a.queue_count_next = 0;
        *a.redo_count_next = 0;
    }
    __syncthreads();

    if (warp == WARPS) {
        // ---- producer: every tile of every piece of this CTA, in order ---------------------------
        if (lane != 0) return;
        const uint64_t pol = l2_evict_first_policy();
        uint32_t i = 0;
        FilterPiece pc;
        for (int k = 0; plan_piece(plan, blockIdx.x, k, pc); ++k) {
            const long long srow = source_row(a, pc.row);
            const bool valid = temp_ok(a.temperature[pc.row / a.G]) && srow >= 0;
            const T* rowp = reinterpret_cast<const T*>(a.logits) + (srow < 0 ? 0 : srow) * a.row_stride;
            for (int ti = pc.tile0; ti < pc.tile1; ++ti, ++i) {
                const int s = (int)(i % STAGES);
                const uint32_t round = i / STAGES;
                if (round > 0) {
                    const int wr = mbar_wait_twice(&empty[s], (round - 1) & 1, wait_limit_ns);
                    if (wr != WAIT_OK) atomicOr(a.status, ST_INTERNAL);
                    if (wr == WAIT_LOST) return;      // nothing more is issued
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
    u64* region = cand + warp * CS_REGION;
    const int region_off = (int)(reinterpret_cast<unsigned char*>(region) - dyn);
    const int hist_off = (int)(reinterpret_cast<unsigned char*>(hist) - dyn);
    // first-tile bound.  k <= 128 (every warp needs at most 16 elements): from the lane maxima, over
    // groups of two or more lanes.  Larger k: the exact need-th largest maximum of groups of g elements,
    // at least 4 k groups in the tile (cheaper bounds from lane maxima or lane pairs let 10 to 25 % of
    // a tile pass: the extra candidates cost more than the search).
    const int need = (k_eff + WARPS - 1) / WARPS;
    int group_lanes = 1;
    while (2 * group_lanes * need <= 32) group_lanes <<= 1;
    int g = VEC;
    while (g > 2 && (TILE_CHUNKS * CHUNK) / g < 4 * k_eff) g >>= 1;

    bool dead = false;      // a wait ran out: this warp computes no more, but takes every tile and joins every barrier
    bool lost = false;      // a wait did not complete at all: the warp stops waiting as well
    uint32_t i = 0;
    int parity = 0;         // which copy of the per-piece state this piece uses
    FilterPiece pc;
    for (int k = 0; plan_piece(plan, blockIdx.x, k, pc); ++k) {
        if (pc.tile0 >= pc.tile1) continue;
        CsShared& cs = css[parity];
        parity ^= 1;
        const int row = pc.row;
        const float Tb = a.temperature[row / a.G];
        const bool in_range = source_row(a, row) >= 0;
        const bool valid = temp_ok(Tb) && in_range;
        const float c32 = temp_scale(Tb);
        float ref_off = 0.f, acc = 0.f;
        int wcount = 0;             // candidates in this warp's region (cs.wcnt[warp] holds the same number)
        int g0 = 0;                 // bin coordinate of the first tile's bound: origin of the histogram
        bool full_region = false;   // the region ran out of room (the row goes to the direct kernel)

        for (int ti = pc.tile0; ti < pc.tile1; ++ti, ++i) {
            const int s = (int)(i % STAGES);
            const uint32_t round = i / STAGES;
            if (!lost) {
                const int wr = mbar_wait_twice(&full[s], round & 1, wait_limit_ns);
                if (wr != WAIT_OK) {
                    dead = true;
                    lost = wr == WAIT_LOST;
                    if (lane == 0) {
                        cta.abort = 1;
                        atomicOr(a.status, ST_INTERNAL);
                    }
                }
            }
            const int c = ti * TILE_CHUNKS + warp;
            const bool work = !dead && valid && !full_region && c < a.nch;
            const unsigned char* chunk = stage_mem + s * TILE_BYTES + warp * (CHUNK * (int)sizeof(T));
            ChunkRegs<T> regs;
            if (work) load_staged(regs, chunk, c * CHUNK, a.V, lane);
            if (ti == pc.tile0 && valid) {
                // first tile of a piece (every warp holds a full chunk): each warp's own bound, then the minimum
                if (work) {
                    unsigned k16;
                    float wm = 0.f;
                    if (SMALL && group_lanes >= 2) {
                        const float lm = regs.lane_max_plain();
                        k16 = first_tile_key_groups(lm, group_lanes);
                        if (STATS) wm = warp_max_redux(lm);
                    } else {
                        k16 = first_tile_key(regs, g, need);
                        if (STATS) wm = warp_max_redux(regs.lane_max_plain());
                    }
                    if (lane == 0) {
                        atomicMin(&cs.thr0_key, k16 << 16);
                        if (STATS && wm == wm) atomicMax(&cs.top_key, orderable(wm));
                    }
                }
                workers_sync();
                const unsigned thr0 = *(volatile unsigned*)&cs.thr0_key;
                g0 = bin_coord(thr0 >> 16);
                if (lane == 0) atomicMax(&cs.thr_key, thr0);
                if (STATS) ref_off = __fmul_rn(from_orderable(*(volatile unsigned*)&cs.top_key), c32);
                __syncwarp();
            }
            int added = 0;          // what this chunk appends to the region
            if (work) {
                const unsigned thr_key = *(volatile unsigned*)&cs.thr_key;
                unsigned mask = pass_mask(regs, thr_of_key(thr_key));
                if (thr_key < 0x00800000u) {
                    // no finite bound (rows of -inf): everything would pass, padding included
                    full_region = true;
                    mask = 0u;
                }
                const int n = __popc(mask);
                added = __reduce_add_sync(0xffffffffu, n);
                if (added) {
                    if (wcount + added > CS_REGION) {
                        // no room: bring the bound up to date and drop what fell below it
                        wcount = maintain_region(wcount, region_off, hist_off, &cs, &cta.wcnt[warp], k_eff);
                        if (wcount + added > CS_REGION) {     // ties, a coarse bin too full, or a very loose bound
                            full_region = true;
                            mask = 0u;
                            added = 0;
                        }
                    }
                    const int vchunk = c * CHUNK;
                    // every lane appends its own passing values: its slots come from the warp's counter
                    if (mask) {
                        int pos = atomicAdd(&cta.wcnt[warp], n);
                        do {
                            const int bit = __ffs(mask) - 1;
                            mask &= mask - 1u;
                            const int off = bit_offset(bit, lane, (const T*)nullptr);
                            const uint32_t bits = __float_as_uint(staged_value(chunk, off, (const T*)nullptr) + 0.0f);   // -0 becomes +0
                            const uint32_t okey = bits ^ ((uint32_t)((int32_t)bits >> 31) | 0x80000000u);
                            region[pos++] = ((u64)okey << 32) | (u64)(~(uint32_t)(vchunk + off));
                        } while (mask);
                    }
                }
            }
            __syncwarp();
            if (lane == 0 && !lost) mbar_arrive(&empty[s]);     // the staged chunk is not read again
            if (work) {
                if (STATS) {
                    acc += lane_exp_sum2(regs, c32, ref_off);
                } else {
                    // without the exp-sum (which turns NaN by itself) a NaN has to be looked for
                    const float lm = regs.lane_max();
                    if (lm != lm) cs.nan = 1;
                }
                // count the new entries in the histogram
                for (int x = wcount + lane; x < wcount + added; x += 32) hist_add(hist, hist_bin((unsigned)(region[x] >> 32), g0));
                wcount += added;
                // the bound is refreshed after every tile, each time by another warp (the others'
                // latest values may not be counted yet, which only makes it a little lower)
                if (warp == (ti & (WARPS - 1))) {
                    __syncwarp();
                    refresh_bound(hist_off, &cs, k_eff);
                }
            }
        }

        // ---- end of the piece: survivors and statistics to the piece's scratch area ------------------
        if (lane == 0 && full_region) cs.overflow = 1;
        if (STATS) {
            const double sw = (double)warp_sum(acc);
            if (lane == 0) cs.wsum[warp] = sw;
        }
        workers_sync();     // every candidate is counted, every flag is set
        const bool piece_ok = valid && !*(volatile int*)&cs.overflow && !*(volatile int*)&cta.abort;
        unsigned thr_final = *(volatile unsigned*)&cs.thr_key;
        if (piece_ok) {
            // the final bound, by every warp for itself (all get the same): no second barrier for it
            const int found = kth_bin(hist, k_eff, lane);
            if (found >= 0) thr_final = max(thr_final, coord_code(g0 + found) << 16);
            // every warp filters its own region and appends to the piece's scratch area
            u64* dst = a.surv_keys + (long long)pc.area * surv_cap;
            const int n = compact_region(region, wcount, thr_final, lane);
            int base = 0;
            if (lane == 0 && n) base = atomicAdd(&cs.m, n);
            base = __shfl_sync(0xffffffffu, base, 0);
            for (int x = lane; x < n; x += 32)
                if (base + x < surv_cap) dst[base + x] = region[x];
        }
        workers_sync();     // the survivors are counted; nobody reads the histogram any more
        if (tid == 0) {
            int flags = 0;
            const int m = cs.m;
            if (cta.abort) flags = CSF_ABORT;
            else if (!in_range) flags = CSF_RANGE;
            else if (!valid) flags = CSF_TEMPERATURE;
            else if (cs.overflow || m > surv_cap) flags = CSF_REDO;      // too many candidates or ties at the bound
            else if (cs.nan) flags = CSF_LOGIT;
            else if (m < k_eff) flags = CSF_REDO;                        // cannot happen with a valid bound; be safe
            double zs = 0.0;
            if (STATS)
                for (int w = 0; w < WARPS; ++w) zs += cs.wsum[w];
            // a reference that later logits overflowed, or NaN / +inf data: the direct kernel sorts it out
            if (STATS && flags == 0 && !(zs > 0.0 && zs < CUDART_INF)) flags = CSF_REDO;
            CsRowMeta meta;
            meta.count = m;
            meta.flags = flags;
            meta.ref_off = ref_off;
            meta.thr_key = thr_final;
            meta.z_stream = zs;
            a.surv_meta[pc.area] = meta;
            cs_reset(cs);       // this copy is used again by the piece after the next one
        }
        // Ready for the next piece, without a barrier of its own: the histogram is not written before
        // the barrier of that piece's first tile, which every warp reaches after its share of this.
        if (lane == 0) cta.wcnt[warp] = 0;
        for (int x = tid; x < CS_HIST_WORDS; x += THREADS) hist[x] = 0u;
    }
}

// ---- block-wide sort in registers ----------------------------------------------------------------
// Bitonic network (descending) over N = 256 * R keys, R per thread: element e = warp * 32R + r * 32
// + lane sits in register r of that lane.  Strides below 32 are warp shuffles, strides 32 .. 16R
// are compare-exchanges between two registers of one thread, and only the three largest strides
// of a merge cross warps: those go through shared memory (two buffers in turn, one barrier per
// stage).  Keys are unsigned and larger = earlier; equal keys are interchangeable.
__device__ __forceinline__ uint32_t shfl_xor_key(uint32_t k, int d) { return __shfl_xor_sync(0xffffffffu, k, d); }
__device__ __forceinline__ u64 shfl_xor_key(u64 k, int d) {
    const uint32_t lo = __shfl_xor_sync(0xffffffffu, (uint32_t)k, d);
    const uint32_t hi = __shfl_xor_sync(0xffffffffu, (uint32_t)(k >> 32), d);
    return ((u64)hi << 32) | lo;
}
template <typename K> __device__ __forceinline__ K key_pick(K mine, K other, bool keep_max) {
    const K hi = mine > other ? mine : other, lo = mine > other ? other : mine;
    return keep_max ? hi : lo;
}

template <typename K, int R>
__device__ __forceinline__ void block_sort_desc(K (&key)[R], K* buf) {
    constexpr int N = THREADS * R;
    const int lane = threadIdx.x & 31;
    const int ebase = (threadIdx.x >> 5) * (32 * R) + lane;
    int phase = 0;
#pragma unroll
    for (int size = 2; size <= N; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            if (stride >= 32 * R) {
                K* bp = buf + (phase & 1) * N;
                ++phase;
#pragma unroll
                for (int r = 0; r < R; ++r) bp[ebase + 32 * r] = key[r];
                __syncthreads();
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const int e = ebase + 32 * r;
                    key[r] = key_pick(key[r], bp[e ^ stride], ((e & size) == 0) == ((e & stride) == 0));
                }
            } else if (stride >= 32) {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const int dr = stride >> 5;
                    if ((r & dr) == 0) {
                        const bool desc = ((ebase + 32 * r) & size) == 0;
                        const K x = key[r], y = key[r + dr];
                        const K hi = x > y ? x : y, lo = x > y ? y : x;
                        key[r] = desc ? hi : lo;
                        key[r + dr] = desc ? lo : hi;
                    }
                }
            } else {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const int e = ebase + 32 * r;
                    key[r] = key_pick(key[r], shfl_xor_key(key[r], stride), ((e & size) == 0) == ((lane & stride) == 0));
                }
            }
        }
    }
}

// Sort `count` keys held in shared memory at in[0 .. count) (the rest of the 256R-element network
// is padding) into out[0 .. 256R), as 64-bit keys, largest first.  `in` may be either exchange
// buffer; out is the first.  NARROW: 16-bit logits whose codes lie in [lo16, lo16 + 2^14) and
// V <= 2^18 run the network on 32-bit keys, (code - lo16) << 18 | index complement.
template <int R, bool NARROW>
__device__ __noinline__ void sort_keys(const u64* in, int count, u64* out, unsigned lo16) {
    const int lane = threadIdx.x & 31;
    const int ebase = (threadIdx.x >> 5) * (32 * R) + lane;
    u64 k[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int e = ebase + 32 * r;
        k[r] = e < count ? in[e] : 0ull;
    }
    __syncthreads();                // every key is in registers: the buffers are free
    if (NARROW) {
        uint32_t n[R];
#pragma unroll
        for (int r = 0; r < R; ++r)
            n[r] = ebase + 32 * r < count ? ((((uint32_t)(k[r] >> 48) - lo16) << 18) | ((uint32_t)k[r] & 0x3FFFFu)) : 0u;
        block_sort_desc<uint32_t, R>(n, reinterpret_cast<uint32_t*>(out));
        __syncthreads();
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const uint32_t o16 = (n[r] >> 18) + lo16;
            // a 16-bit logit's orderable form ends in sixteen ones when the logit is negative
            const uint32_t o32 = (o16 << 16) | ((o16 & 0x8000u) ? 0u : 0xFFFFu);
            out[ebase + 32 * r] = ((u64)o32 << 32) | (u64)(0xFFFC0000u | (n[r] & 0x3FFFFu));
        }
    } else {
        block_sort_desc<u64, R>(k, out);
        __syncthreads();
#pragma unroll
        for (int r = 0; r < R; ++r) out[ebase + 32 * r] = k[r];
    }
    __syncthreads();
}

constexpr int CS_TIE_CAP = 256;     // boundary-group size up to which the survivors are trimmed to k
constexpr int CS_MAX_PIECES = 8;    // most pieces a row is dealt in

struct CsFinishShared {
    unsigned hi16;      // largest 16-bit logit code among the survivors
    int kept, ties;     // slot counters: survivors above the bound's code / with it
    int overflow;       // more survivors than the exchange buffers hold
    int found;          // multi-piece rows: bin of the k-th largest code among all pieces' survivors
    int piece_id[CS_MAX_PIECES];
    int piece_count[CS_MAX_PIECES];
};

// One CTA per row: put the row's pieces together, trim the survivors to the k best where that is
// cheap, sort, cut / renormalise / emit.  The survivors of a piece are all its elements at or above
// its final bound, i.e. its k best plus whatever shares the bound's 16-bit code with the k-th (ties
// of a 16-bit logit; values within 2^-7 relative of it for 32-bit logits).  The largest of the
// pieces' bounds is a bound for the row.  A row in several pieces holds about k survivors per piece
// above it: their 16-bit codes are counted in the filter kernel's two-level histogram first, which
// gives the code of the row's k-th largest logit, and only survivors at or above that code go on.
// When the survivors would need a larger sort network than k keys do, the members of the boundary
// group (the lowest code) are ranked among themselves (all pairs) and only the best
// k - (number above the group) are kept.
template <typename T, bool STATS>
__global__ void __launch_bounds__(THREADS, 6) compress_finish_kernel(CompressArgs a, FilterPlan plan, int n2cap) {
    extern __shared__ u64 keys[];          // two exchange buffers of n2cap keys; the sorted keys end up in the first
    __shared__ CompressShared sh;
    __shared__ CsFinishShared fs;
    __shared__ __align__(16) unsigned fhist[CS_HIST_WORDS];    // (kth_bin reads four super-bins at a time)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row = blockIdx.x;
    int k_eff = a.top_k > 0 ? a.top_k : a.k_max;
    if (k_eff > a.k_max) k_eff = a.k_max;
    if (k_eff > a.V) k_eff = a.V;
    const int surv_cap = cs_survivor_cap(a.k_max);
    // the scratch areas that hold this row: its own, or those of its pieces if it was dealt in pieces
    const int whole_rows = plan.q * plan.grid;
    const bool split_row = row >= whole_rows;
    const int area0 = split_row ? plan.rows + (row - whole_rows) * plan.split : row;
    const int nareas = split_row ? plan.split : 1;
    grid_dependency_sync();
    // the first piece's first 512 scratch slots exist for every k_max: requested before its count is known
    const u64* src0 = a.surv_keys + (long long)area0 * surv_cap;
    const u64 first0 = src0[tid], first1 = src0[tid + THREADS];
    // ---- the pieces: flags, the row's bound ----------------------------------------------------------
    int np = 0, flags = 0;
    unsigned thr_key = 0u;
    for (int j = 0; j < nareas; ++j) {
        if (split_row && j > 0 && plan_piece_tile(plan, j + 1) <= plan_piece_tile(plan, j)) continue;   // an empty piece
        const CsRowMeta meta = a.surv_meta[area0 + j];
        flags |= meta.flags;
        thr_key = max(thr_key, meta.thr_key);
        if (np < CS_MAX_PIECES && tid == 0) {
            fs.piece_id[np] = area0 + j;
            fs.piece_count[np] = meta.count;
        }
        ++np;
    }
    if (np > CS_MAX_PIECES) flags |= CSF_REDO;
    if (flags & (CSF_ABORT | CSF_TEMPERATURE | CSF_LOGIT | CSF_RANGE)) {
        emit_invalid_row(a, row);
        if (tid == 0 && !(flags & CSF_ABORT))
            atomicOr(a.status, (flags & CSF_TEMPERATURE) ? ST_TEMPERATURE : (flags & CSF_RANGE) ? ST_RANGE : ST_LOGIT);
        return;
    }
    if (flags & CSF_REDO) {
        // a piece's candidates did not fit: the direct kernel writes this row
        if (tid == 0) {
            a.redo_rows[atomicAdd(a.redo_count, 1)] = row;
            atomicAdd(a.redo_total, 1ull);
        }
        return;
    }
    const float Tb = a.temperature[row / a.G];
    u64* bufA = keys;
    u64* bufB = keys + n2cap;
    if (tid == 0) {
        fs.hi16 = 0u;
        fs.kept = 0;
        fs.ties = 0;
        fs.overflow = 0;
        fs.found = -1;
    }
    if (np > 1)
        for (int x = tid; x < CS_HIST_WORDS; x += THREADS) fhist[x] = 0u;
    __syncthreads();
    if (np > 1) {
        // ---- several pieces: the code of the row's k-th largest logit among all their survivors ------
        const int g0 = bin_coord(thr_key >> 16);
        for (int p = 0; p < np; ++p) {
            const u64* src = a.surv_keys + (long long)fs.piece_id[p] * surv_cap;
            const int m = fs.piece_count[p];
            for (int e = tid; e < m; e += THREADS) {
                const unsigned okey = (unsigned)(src[e] >> 32);
                if (okey >= thr_key) hist_add(fhist, hist_bin(okey, g0));
            }
        }
        __syncthreads();
        if (warp == 0) {
            const int found = kth_bin(fhist, k_eff, lane);
            if (lane == 0) fs.found = found;
        }
        __syncthreads();
        if (fs.found >= 0) thr_key = max(thr_key, coord_code(g0 + fs.found) << 16);
    }
    const unsigned thr16 = thr_key >> 16;
    // ---- survivors to shared memory: those above the bound's code to buffer A, the boundary group
    // ---- to buffer B, both in arrival order (warp-aggregated slots)
    {
        const unsigned lt = (1u << lane) - 1u;
        unsigned hi = 0u;
        for (int p = 0; p < np; ++p) {
            const u64* src = a.surv_keys + (long long)fs.piece_id[p] * surv_cap;
            const int m = fs.piece_count[p];
            for (int e0 = 0; e0 < m; e0 += THREADS) {
                const int e = e0 + tid;
                const u64 key = (p == 0 && e0 == 0) ? first0 : (p == 0 && e0 == THREADS) ? first1 : (e < m ? src[e] : 0ull);
                const unsigned code = (unsigned)(key >> 48);
                const bool live = e < m && (unsigned)(key >> 32) >= thr_key;
                const bool is_above = live && code > thr16;
                const bool is_tie = live && !is_above;
                if (live) hi = max(hi, code);
                const unsigned ma = __ballot_sync(0xffffffffu, is_above), mt = __ballot_sync(0xffffffffu, is_tie);
                int ba = 0, bt = 0;
                if (lane == 0) {
                    if (ma) ba = atomicAdd(&fs.kept, __popc(ma));
                    if (mt) bt = atomicAdd(&fs.ties, __popc(mt));
                }
                ba = __shfl_sync(0xffffffffu, ba, 0);
                bt = __shfl_sync(0xffffffffu, bt, 0);
                const int sa = ba + __popc(ma & lt), st = bt + __popc(mt & lt);
                if (is_above) {
                    if (sa < n2cap) bufA[sa] = key;
                    else fs.overflow = 1;
                }
                if (is_tie) {
                    if (st < n2cap) bufB[st] = key;
                    else fs.overflow = 1;
                }
            }
        }
        hi = __reduce_max_sync(0xffffffffu, hi);
        if (lane == 0) atomicMax(&fs.hi16, hi);
    }
    __syncthreads();
    const int above = fs.kept, t = fs.ties, m = above + t;
    if (fs.overflow || m > n2cap || m < k_eff) {
        // more survivors than the buffers hold (a histogram window too coarse for this row): direct kernel
        if (tid == 0) {
            a.redo_rows[atomicAdd(a.redo_count, 1)] = row;
            atomicAdd(a.redo_total, 1ull);
        }
        return;
    }
    const bool narrow = sizeof(T) == 2 && a.V <= (1 << 18) && fs.hi16 - thr16 < (1u << 14);
    int nk = 256;                       // network size for k keys
    while (nk < k_eff) nk <<= 1;
    int nm = 256;                       // network size for all m survivors
    while (nm < m) nm <<= 1;
    int count = m, n2 = nm;
    if (nm > nk && above < k_eff && t <= CS_TIE_CAP) {
        // trim: of the boundary group only the best k - above, each placed by its rank in the group
        const int need = k_eff - above;
        for (int j = tid; j < t; j += THREADS) {
            const u64 key = bufB[j];
            int rank = 0;
            for (int x = 0; x < t; ++x) rank += bufB[x] > key ? 1 : 0;
            if (rank < need) bufA[above + rank] = key;      // keys are distinct: every rank is taken once
        }
        count = k_eff;
        n2 = nk;
    } else {
        for (int j = tid; j < t; j += THREADS) bufA[above + j] = bufB[j];
    }
    __syncthreads();
    const u64* in = bufA;
    // the boundary group's ranks are written (or nothing was): sort `count` keys from `in`
    // (sort_keys moves them to registers before either buffer is reused)
    const int R = n2 >> 8;
    if (narrow) {
        if (R == 1) sort_keys<1, true>(in, count, bufA, thr16);
        else if (R == 2) sort_keys<2, true>(in, count, bufA, thr16);
        else if (R == 4) sort_keys<4, true>(in, count, bufA, thr16);
        else sort_keys<8, true>(in, count, bufA, thr16);
    } else {
        if (R == 1) sort_keys<1, false>(in, count, bufA, 0u);
        else if (R == 2) sort_keys<2, false>(in, count, bufA, 0u);
        else if (R == 4) sort_keys<4, false>(in, count, bufA, 0u);
        else sort_keys<8, false>(in, count, bufA, 0u);
    }
    const float top = key_logit(keys[0]);
    double Z = 0.0;
    if (STATS) {
        // move every piece's streamed sum from its reference onto the scale of the weights exp(l/T - top/T)
        const float c32 = temp_scale(Tb);
        for (int p = 0; p < np; ++p) {
            const CsRowMeta meta = a.surv_meta[fs.piece_id[p]];
            Z += meta.z_stream * exp2((double)meta.ref_off - (double)top * (double)c32);
        }
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
