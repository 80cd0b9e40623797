// C-ABI of the picospec library: context, argument checks, kernel launches.  See picospec.h.
#include "../../include/picospec.h"

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>

#include <mutex>

#include "compress_kernels.cuh"
#include "compress_stream_kernel.cuh"
#include "verify_kernels.cuh"
#include "edge_kernels.cuh"
#include "wire_kernels.cuh"
#include "vocab_parallel_kernels.cuh"

using namespace picospec;

#define PROF_RING 128
// most CTAs per SM any shape of the staged filter kernel runs at (sizes the per-piece scratch)
#define FILTER_MAX_CTAS_PER_SM 4

struct picospec_ctx {
    int device;
    int max_batch, max_gamma, max_vocab, max_k;
    int num_sms;
    unsigned long long wait_limit_ns;   // first limit of the staged kernels' waits
    int last_cuda_error;
    unsigned long long compress_calls;
    // optional per-kernel timing (picospec_profile_*): rings of event pairs per kernel kind
    int prof_level;
    cudaEvent_t prof_ev[PICOSPEC_PROF_KINDS][PROF_RING][2];
    long long prof_count[PICOSPEC_PROF_KINDS];
    int prof_every;                                   // bracket every prof_every-th launch of a kind
    long long prof_seq[PICOSPEC_PROF_KINDS];
    // workspace
    float2* stats;
    double* dsum;
    float* row_max;
    int* queue;
    unsigned long long* need_rows;
    int* counters;  // [0] verify queue, [1],[2] compress queue (alternating), [3],[4] compress redo list (alternating)
    int* redo_rows; // rows the staged compress kernel hands to the direct kernel
    unsigned long long* surv_keys;  // staged compress: survivors per row
    CsRowMeta* surv_meta;
    int* wire_off;                  // wire codec: first entry of each row, [rows + 1]
    int* vp_listed;                 // vocabulary-parallel verify: per sequence, its kind in the double-precision pass
    int* tickets;                   // compress: per queue slot, chunk sums completed in the double-precision cut
    int* rowq;                      // verify: rows whose exact chunk sums are wanted (count: counters[5])
    long long max_rows;
    unsigned* status;
    unsigned long long* slow_rows;
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) ok = false;
        if (ok && prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        target = dev;
    }
    ~DeviceGuard() {
        if (prev >= 0 && prev != target) cudaSetDevice(prev);
    }
    int target;
};

// Brackets one kernel launch with a pair of events when profiling is enabled for its kind.
struct ProfScope {
    picospec_ctx* ctx;
    int kind;
    cudaStream_t s;
    bool on;
    ProfScope(picospec_ctx* c, int k, int min_level, cudaStream_t st) : ctx(c), kind(k), s(st) {
        on = c->prof_level >= min_level;
        if (on) on = (c->prof_seq[k]++ % c->prof_every) == 0;
        if (on) cudaEventRecord(c->prof_ev[k][c->prof_count[k] % PROF_RING][0], s);
    }
    ~ProfScope() {
        if (on) {
            cudaEventRecord(ctx->prof_ev[kind][ctx->prof_count[kind] % PROF_RING][1], s);
            ctx->prof_count[kind]++;
        }
    }
};

int fail_cuda(picospec_ctx* ctx, cudaError_t e) {
    if (ctx) ctx->last_cuda_error = (int)e;
    return PICOSPEC_ECUDA;
}

bool rows_aligned(const void* base, long long row_stride, int elem) {
    return ((uintptr_t)base % 16 == 0) && ((row_stride * elem) % 16 == 0);
}

template <typename T> void set_compress_attrs() {
    cudaFuncSetAttribute(compress_kernel<T, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, COMPRESS_SMEM);
    cudaFuncSetAttribute(compress_kernel<T, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, COMPRESS_SMEM);
    cudaFuncSetAttribute(compress_kernel<T, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, COMPRESS_SMEM);
    cudaFuncSetAttribute(compress_kernel<T, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, COMPRESS_SMEM);
}

template <typename T> cudaError_t set_filter_attrs() {
    cudaError_t e = cudaFuncSetAttribute(compress_filter_kernel<T, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         CsGeom<T, true>::SMEM_BYTES);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(compress_filter_kernel<T, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 CsGeom<T, true>::SMEM_BYTES);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(compress_filter_kernel<T, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 CsGeom<T, false>::SMEM_BYTES);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(compress_filter_kernel<T, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 CsGeom<T, false>::SMEM_BYTES);
    return e;
}

// Opt-in shared-memory sizes of the staged kernels: once per device and process.
cudaError_t ensure_kernel_attrs(int device) {
    static std::mutex mu;
    static bool done[64];
    if (device < 0 || device >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (done[device]) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(chunk_stats_bulk_kernel<__nv_bfloat16>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         TileGeom<__nv_bfloat16>::SMEM_BYTES);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(chunk_stats_bulk_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 TileGeom<float>::SMEM_BYTES);
    if (e == cudaSuccess) e = set_filter_attrs<__nv_bfloat16>();
    if (e == cudaSuccess) e = set_filter_attrs<float>();
    if (e == cudaSuccess) done[device] = true;
    return e;
}

// Launch with programmatic stream serialization: the kernel's CTAs may be scheduled while the
// kernel before it in the stream drains (every kernel starts with grid_dependency_sync()).
// Launch errors are picked up by the callers through cudaGetLastError().
template <typename... P, typename... A>
void launch_chained(void (*kern)(P...), int grid, int block, size_t smem, cudaStream_t s, A&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    (void)cudaLaunchKernelEx(&cfg, kern, static_cast<P>(args)...);
}

template <typename T, bool ALIGNED>
void launch_compress_direct(const CompressArgs& a, int grid, bool stats, cudaStream_t s) {
    if (stats) launch_chained(compress_kernel<T, ALIGNED, true>, grid, THREADS, COMPRESS_SMEM, s, a);
    else launch_chained(compress_kernel<T, ALIGNED, false>, grid, THREADS, COMPRESS_SMEM, s, a);
}

template <typename T>
cudaError_t launch_compress(picospec_ctx* ctx, const CompressArgs& a, bool aligned, cudaStream_t s) {
    const int rows = a.B * a.G;
    const int grid = rows < ctx->num_sms * 2 ? rows : ctx->num_sms * 2;
    const bool stats = a.top_p < 1.0f || a.raw_probs;     // raw probabilities need the normaliser too
    // staged kernel: 16-byte aligned rows of at least one full tile
    const bool staged = aligned && ((size_t)a.V * sizeof(T)) % 16 == 0 && a.V >= TILE_CHUNKS * CHUNK;
    if (staged) {
        cudaError_t ea = ensure_kernel_attrs(ctx->device);
        if (ea != cudaSuccess) return ea;
        int k_eff = a.top_k > 0 ? a.top_k : a.k_max;
        if (k_eff > a.k_max) k_eff = a.k_max;
        const bool small = k_eff <= CS_K_SMALL;
        void (*kern)(CompressArgs, FilterPlan, unsigned long long) =
            small ? (stats ? compress_filter_kernel<T, true, true> : compress_filter_kernel<T, false, true>)
                  : (stats ? compress_filter_kernel<T, true, false> : compress_filter_kernel<T, false, false>);
        const int smem = small ? CsGeom<T, true>::SMEM_BYTES : CsGeom<T, false>::SMEM_BYTES;
        int per_sm = 1;     // resident CTAs per SM for this kernel's registers and shared memory
        cudaError_t eo = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, STREAM_THREADS, smem);
        if (eo != cudaSuccess) return eo;
        if (per_sm < 1) per_sm = 1;
        if (per_sm > FILTER_MAX_CTAS_PER_SM) per_sm = FILTER_MAX_CTAS_PER_SM;
        // whole rows first, the remainder in pieces so that every CTA streams about the same number of tiles
        const FilterPlan plan = make_filter_plan(rows, (a.nch + TILE_CHUNKS - 1) / TILE_CHUNKS,
                                                 a.V % (TILE_CHUNKS * CHUNK) != 0, (long long)ctx->num_sms * per_sm);
        {
            ProfScope ps(ctx, PICOSPEC_PROF_COMPRESS_STREAM, 1, s);
            launch_chained(kern, plan.grid, STREAM_THREADS, smem, s, a, plan, ctx->wait_limit_ns);
        }
        cudaError_t e0 = cudaGetLastError();
        if (e0 != cudaSuccess) return e0;
        {
            int n2 = 1;
            while (n2 < cs_survivor_cap(a.k_max)) n2 <<= 1;
            ProfScope ps(ctx, PICOSPEC_PROF_COMPRESS_FINISH, 2, s);
            // two exchange buffers of the sort network (the sorted keys end up in the first)
            if (stats) launch_chained(compress_finish_kernel<T, true>, rows, THREADS, (size_t)n2 * 16, s, a, plan, n2);
            else launch_chained(compress_finish_kernel<T, false>, rows, THREADS, (size_t)n2 * 16, s, a, plan, n2);
        }
        e0 = cudaGetLastError();
        if (e0 != cudaSuccess) return e0;
        // rows whose candidates did not fit (normally none: every CTA returns at once)
        CompressArgs r = a;
        r.use_redo_list = 1;
        ProfScope ps(ctx, PICOSPEC_PROF_COMPRESS_REDO, 2, s);
        launch_compress_direct<T, true>(r, grid, stats, s);
    } else {
        ProfScope ps(ctx, PICOSPEC_PROF_COMPRESS_STREAM, 1, s);
        if (aligned) launch_compress_direct<T, true>(a, grid, stats, s);
        else launch_compress_direct<T, false>(a, grid, stats, s);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || !stats) return e;
    ProfScope ps2(ctx, PICOSPEC_PROF_COMPRESS_PRECISE, 2, s);
    // rows whose top-p cut was too close to call: exact normaliser, then redo the cut
    PreciseArgs p;
    p.logits = a.logits; p.row_stride = a.row_stride; p.V = a.V; p.nch = a.nch;
    p.seq_rows = a.G; p.temperature = a.temperature;
    p.rows = a.queue; p.row_count = a.queue_count; p.row_max = a.row_max; p.dsum = a.dsum;
    // exact sums and the cut of the queued rows in one kernel
    launch_chained(compress_precise_kernel<T>, ctx->num_sms * 6, THREADS, MAX_K * 8, s, a, p);
    return cudaGetLastError();
}

// the streaming statistics pass over the rows a call reads
template <typename T>
cudaError_t launch_verify_stream(picospec_ctx* ctx, const VerifyArgs& a, bool aligned, cudaStream_t s) {
    const int stream_rows = a.sample_only ? a.B : a.B * (a.r1 - a.r0);
    const long long items = (long long)stream_rows * a.nch;
    long long want = (items + WARPS - 1) / WARPS;
    const int cap = ctx->num_sms * 4;
    const int grid = (int)(want < cap ? want : cap);
    const bool staged = aligned && ((size_t)a.V * sizeof(T)) % 16 == 0;
    if (staged) {
        cudaError_t ea = ensure_kernel_attrs(ctx->device);
        if (ea != cudaSuccess) return ea;
        const int tiles_per_row = (a.nch + TileGeom<T>::CHUNKS - 1) / TileGeom<T>::CHUNKS;
        const long long tiles = (long long)stream_rows * tiles_per_row;
        const int gcap = ctx->num_sms * StreamCfg<T>::CTAS_PER_SM;
        const int g = (int)(tiles < gcap ? tiles : gcap);
        ProfScope ps(ctx, PICOSPEC_PROF_VERIFY_STREAM, 1, s);
        launch_chained(chunk_stats_bulk_kernel<T>, g, STREAM_THREADS, TileGeom<T>::SMEM_BYTES, s, a, tiles_per_row, tiles,
                       ctx->wait_limit_ns);
    } else {
        ProfScope ps(ctx, PICOSPEC_PROF_VERIFY_STREAM, 1, s);
        if (aligned) launch_chained(chunk_stats_kernel<T, true>, grid, THREADS, 0, s, a);
        else launch_chained(chunk_stats_kernel<T, false>, grid, THREADS, 0, s, a);
    }
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_verify(picospec_ctx* ctx, const VerifyArgs& a, bool aligned, cudaStream_t s, bool edge = false) {
    {
        cudaError_t e0 = launch_verify_stream<T>(ctx, a, aligned, s);
        if (e0 != cudaSuccess) return e0;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const size_t dyn = (size_t)a.nch * sizeof(double);
    {
        ProfScope ps(ctx, PICOSPEC_PROF_VERIFY_FINISH, 2, s);
        if (edge) launch_chained(edge_finish_kernel<T, false>, a.B, THREADS, 0, s, a);
        else launch_chained(verify_finish_kernel<T, false>, a.B, THREADS, dyn, s, a);
    }
    ProfScope ps3(ctx, PICOSPEC_PROF_VERIFY_PRECISE, 2, s);
    PreciseArgs p;
    p.logits = a.logits; p.row_stride = a.row_stride; p.V = a.V; p.nch = a.nch;
    p.seq_rows = a.G + 1; p.temperature = a.temperature;
    p.rows = a.rowq; p.row_count = a.rowq_count;
    p.row_max = a.row_max; p.dsum = a.dsum;
    launch_chained(precise_chunk_sums_kernel<T>, ctx->num_sms * 6, THREADS, 0, s, p);
    const int g2 = a.B < ctx->num_sms ? a.B : ctx->num_sms;
    if (edge) launch_chained(edge_finish_kernel<T, true>, g2, THREADS, 0, s, a);
    else launch_chained(verify_finish_kernel<T, true>, g2, THREADS, dyn, s, a);
    return cudaGetLastError();
}

// workspace pointers and the alternating counters of one compress-type call
void fill_compress_workspace(picospec_ctx* ctx, CompressArgs& a) {
    a.row_max = ctx->row_max; a.dsum = ctx->dsum; a.queue = ctx->queue;
    const int cur = 1 + (int)(ctx->compress_calls & 1ull);
    a.queue_count = ctx->counters + cur;
    a.queue_count_next = ctx->counters + (3 - cur);
    a.tickets = ctx->tickets;
    a.redo_rows = ctx->redo_rows;
    a.redo_count = ctx->counters + 2 + cur;           // [3] / [4]
    a.redo_count_next = ctx->counters + 2 + (3 - cur);
    a.use_redo_list = 0;
    a.redo_total = ctx->slow_rows + 1;
    a.surv_keys = ctx->surv_keys;
    a.surv_meta = ctx->surv_meta;
    ctx->compress_calls++;
    a.status = ctx->status; a.slow_rows = ctx->slow_rows;
}

int check_common(const picospec_ctx* ctx, const void* logits, int dtype, int B, int G, int V, long long row_stride,
                 const float* temperature, int k_max) {
    if (!ctx || !logits || !temperature) return PICOSPEC_EINVAL;
    if (dtype != PICOSPEC_F32 && dtype != PICOSPEC_BF16) return PICOSPEC_EINVAL;
    if (B < 0 || G < 0 || V <= 0 || k_max <= 0 || row_stride < V) return PICOSPEC_EINVAL;
    if (B > ctx->max_batch || G > ctx->max_gamma || V > ctx->max_vocab || k_max > ctx->max_k)
        return PICOSPEC_ECAPACITY;
    return PICOSPEC_OK;
}

}  // namespace

extern "C" {

int picospec_create(picospec_ctx** out, int device, int max_batch, int max_gamma, int max_vocab, int max_k) {
    if (!out) return PICOSPEC_EINVAL;
    *out = nullptr;
    if (device < 0 || max_batch <= 0 || max_gamma < 0 || max_gamma > PICOSPEC_MAX_GAMMA || max_vocab <= 0 ||
        max_vocab > (1 << 22) || max_k <= 0 || max_k > PICOSPEC_MAX_K)
        return PICOSPEC_EINVAL;
    picospec_ctx* ctx = (picospec_ctx*)calloc(1, sizeof(picospec_ctx));
    if (!ctx) return PICOSPEC_EINVAL;
    ctx->device = device;
    ctx->max_batch = max_batch;
    ctx->max_gamma = max_gamma;
    ctx->max_vocab = max_vocab;
    ctx->max_k = max_k;
    ctx->wait_limit_ns = WAIT_LIMIT_NS;
    DeviceGuard g(device);
    cudaError_t e = g.ok ? cudaSuccess : cudaErrorInvalidDevice;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, device);
    const size_t rows = (size_t)max_batch * (max_gamma + 1);
    const size_t nch = ((size_t)max_vocab + CHUNK - 1) / CHUNK;
    if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->stats, rows * nch * sizeof(float2));
    if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->dsum, rows * nch * sizeof(double));
    if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->row_max, rows * sizeof(float));
    if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->queue, rows * sizeof(int));
    if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->need_rows, rows * sizeof(unsigned long long));
    if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->counters, 8 * sizeof(int));
    if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->redo_rows, rows * sizeof(int));
    // one scratch area per whole row and per piece of a row that is dealt in pieces (at most twice
    // the CTAs of the filter kernel)
    const size_t pieces = rows + 2 * (size_t)ctx->num_sms * FILTER_MAX_CTAS_PER_SM;
    if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->surv_keys, pieces * (size_t)cs_survivor_cap(max_k) * sizeof(unsigned long long));
    if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->surv_meta, pieces * sizeof(CsRowMeta));
    if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->wire_off, (rows + 1) * sizeof(int));
    if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->vp_listed, (size_t)max_batch * sizeof(int));
    if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->tickets, rows * sizeof(int));
    if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->rowq, rows * sizeof(int));
    ctx->max_rows = (long long)rows;
    if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->status, sizeof(unsigned));
    if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->slow_rows, 2 * sizeof(unsigned long long));   // [0] slow rows, [1] redo rows
    if (e == cudaSuccess) e = cudaMemset(ctx->counters, 0, 8 * sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(ctx->status, 0, sizeof(unsigned));
    if (e == cudaSuccess) e = cudaMemset(ctx->slow_rows, 0, 2 * sizeof(unsigned long long));
    if (e == cudaSuccess) {
        set_compress_attrs<float>();
        set_compress_attrs<__nv_bfloat16>();
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) {
        picospec_destroy(ctx);
        return PICOSPEC_ECUDA;
    }
    *out = ctx;
    return PICOSPEC_OK;
}

int picospec_destroy(picospec_ctx* ctx) {
    if (!ctx) return PICOSPEC_EINVAL;
    DeviceGuard g(ctx->device);
    picospec_profile_enable(ctx, 0);
    cudaFree(ctx->stats);
    cudaFree(ctx->dsum);
    cudaFree(ctx->row_max);
    cudaFree(ctx->queue);
    cudaFree(ctx->need_rows);
    cudaFree(ctx->counters);
    cudaFree(ctx->redo_rows);
    cudaFree(ctx->surv_keys);
    cudaFree(ctx->surv_meta);
    cudaFree(ctx->wire_off);
    cudaFree(ctx->vp_listed);
    cudaFree(ctx->tickets);
    cudaFree(ctx->rowq);
    cudaFree(ctx->status);
    cudaFree(ctx->slow_rows);
    free(ctx);
    return PICOSPEC_OK;
}

const char* picospec_strerror(int err) {
    switch (err) {
        case PICOSPEC_OK: return "ok";
        case PICOSPEC_EINVAL: return "invalid argument";
        case PICOSPEC_ECUDA: return "CUDA runtime error";
        case PICOSPEC_ECAPACITY: return "problem size exceeds the context's capacity";
        case PICOSPEC_EDATA: return "a kernel found bad data (see the status word)";
        default: return "unknown error";
    }
}

int picospec_last_cuda_error(const picospec_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }

int picospec_wait_limit(picospec_ctx* ctx, unsigned long long limit_ns) {
    if (!ctx) return PICOSPEC_EINVAL;
    ctx->wait_limit_ns = limit_ns < WAIT_LIMIT_NS ? limit_ns : WAIT_LIMIT_NS;
    return PICOSPEC_OK;
}

int picospec_profile_enable(picospec_ctx* ctx, int level) {
    if (!ctx || level < 0 || level > 2) return PICOSPEC_EINVAL;
    DeviceGuard g(ctx->device);
    const bool have = ctx->prof_ev[0][0][0] != nullptr;
    if (level > 0 && !have) {
        for (int k = 0; k < PICOSPEC_PROF_KINDS; ++k)
            for (int i = 0; i < PROF_RING; ++i)
                for (int j = 0; j < 2; ++j) {
                    cudaError_t e = cudaEventCreate(&ctx->prof_ev[k][i][j]);
                    if (e != cudaSuccess) return fail_cuda(ctx, e);
                }
    }
    if (level == 0 && have) {
        for (int k = 0; k < PICOSPEC_PROF_KINDS; ++k)
            for (int i = 0; i < PROF_RING; ++i)
                for (int j = 0; j < 2; ++j) {
                    cudaEventDestroy(ctx->prof_ev[k][i][j]);
                    ctx->prof_ev[k][i][j] = nullptr;
                }
    }
    for (int k = 0; k < PICOSPEC_PROF_KINDS; ++k) ctx->prof_count[k] = ctx->prof_seq[k] = 0;
    ctx->prof_level = level;
    if (ctx->prof_every < 1) ctx->prof_every = 1;
    return PICOSPEC_OK;
}

int picospec_profile_period(picospec_ctx* ctx, int every) {
    if (!ctx || every < 1) return PICOSPEC_EINVAL;
    ctx->prof_every = every;
    for (int k = 0; k < PICOSPEC_PROF_KINDS; ++k) ctx->prof_seq[k] = 0;
    return PICOSPEC_OK;
}

int picospec_profile_read(picospec_ctx* ctx, int kind, float* total_ms_out, int* launches_out, void* cuda_stream) {
    if (!ctx || kind < 0 || kind >= PICOSPEC_PROF_KINDS || !total_ms_out || !launches_out) return PICOSPEC_EINVAL;
    DeviceGuard g(ctx->device);
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)cuda_stream);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    const long long n = ctx->prof_count[kind] < PROF_RING ? ctx->prof_count[kind] : PROF_RING;
    float total = 0.f;
    for (long long i = 0; i < n; ++i) {
        float ms = 0.f;
        e = cudaEventElapsedTime(&ms, ctx->prof_ev[kind][i][0], ctx->prof_ev[kind][i][1]);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
        total += ms;
    }
    *total_ms_out = total;
    *launches_out = (int)n;
    ctx->prof_count[kind] = 0;
    return PICOSPEC_OK;
}

int picospec_profile_samples(picospec_ctx* ctx, int kind, float* ms_out, int capacity, int* n_out, void* cuda_stream) {
    if (!ctx || kind < 0 || kind >= PICOSPEC_PROF_KINDS || !ms_out || !n_out || capacity < 0) return PICOSPEC_EINVAL;
    DeviceGuard g(ctx->device);
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)cuda_stream);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    const long long total = ctx->prof_count[kind];
    long long n = total < PROF_RING ? total : PROF_RING;
    if (n > capacity) n = capacity;
    // the ring holds the last PROF_RING brackets; the newest n of them, oldest first
    for (long long i = 0; i < n; ++i) {
        const long long slot = (total - n + i) % PROF_RING;
        float ms = 0.f;
        e = cudaEventElapsedTime(&ms, ctx->prof_ev[kind][slot][0], ctx->prof_ev[kind][slot][1]);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
        ms_out[i] = ms;
    }
    *n_out = (int)n;
    ctx->prof_count[kind] = 0;
    return PICOSPEC_OK;
}

int picospec_status(picospec_ctx* ctx, int* device_status_out, long long* slow_path_rows_out, int clear,
                    void* cuda_stream) {
    if (!ctx) return PICOSPEC_EINVAL;
    DeviceGuard g(ctx->device);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    unsigned st = 0;
    unsigned long long slow = 0;
    cudaError_t e = cudaMemcpyAsync(&st, ctx->status, sizeof(st), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(&slow, ctx->slow_rows, sizeof(slow), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && clear) {
        e = cudaMemsetAsync(ctx->status, 0, sizeof(unsigned), s);
        if (e == cudaSuccess) e = cudaMemsetAsync(ctx->slow_rows, 0, sizeof(unsigned long long), s);
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    if (device_status_out) *device_status_out = (int)st;
    if (slow_path_rows_out) *slow_path_rows_out = (long long)slow;
    return st ? PICOSPEC_EDATA : PICOSPEC_OK;
}

int picospec_counters(picospec_ctx* ctx, long long* out, int clear, void* cuda_stream) {
    if (!ctx || !out) return PICOSPEC_EINVAL;
    DeviceGuard g(ctx->device);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    unsigned long long v[2] = {0, 0};
    cudaError_t e = cudaMemcpyAsync(v, ctx->slow_rows, sizeof(v), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && clear) e = cudaMemsetAsync(ctx->slow_rows, 0, sizeof(v), s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    out[0] = (long long)v[0];
    out[1] = (long long)v[1];
    return PICOSPEC_OK;
}

long long picospec_wire_bytes(int rows, long long entries, int prob_type) {
    if (rows < 0 || entries < 0 || (prob_type != 0 && prob_type != 1)) return -1;
    return wire_bytes(rows, entries, prob_type);
}

static int wire_common(picospec_ctx* ctx, WireArgs& a, bool pack, void* cuda_stream) {
    if (!ctx || !a.q_idx || !a.q_prob || !a.q_count || !a.buf) return PICOSPEC_EINVAL;
    if (a.R < 0 || a.K <= 0 || a.K > PICOSPEC_MAX_K || a.capacity < 0) return PICOSPEC_EINVAL;
    if (pack && (a.prob_type != 0 && a.prob_type != 1)) return PICOSPEC_EINVAL;
    if (((uintptr_t)a.buf & 3u) != 0) return PICOSPEC_EINVAL;
    if (a.R > ctx->max_rows) return PICOSPEC_ECAPACITY;
    if (a.R == 0 && !pack) return PICOSPEC_OK;
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail_cuda(ctx, cudaErrorInvalidDevice);
    a.offsets = ctx->wire_off;
    a.status = ctx->status;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const int rows_grid = a.R > 0 ? (a.R + WARPS - 1) / WARPS : 1;
    const int grid = rows_grid < ctx->num_sms * 8 ? rows_grid : ctx->num_sms * 8;
    if (pack) {
        launch_chained(wire_scan_kernel<true>, 1, THREADS, 0, s, a);
        launch_chained(wire_move_kernel<true>, grid, THREADS, 0, s, a);
    } else {
        launch_chained(wire_scan_kernel<false>, 1, THREADS, 0, s, a);
        launch_chained(wire_move_kernel<false>, grid, THREADS, 0, s, a);
    }
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? PICOSPEC_OK : fail_cuda(ctx, e);
}

int picospec_wire_pack(picospec_ctx* ctx, const int* q_idx, const float* q_prob, const int* q_count, int rows, int k,
                       int prob_type, void* buf, long long capacity_bytes, long long* bytes_out, void* cuda_stream) {
    if (!bytes_out) return PICOSPEC_EINVAL;
    WireArgs a;
    a.q_idx = const_cast<int*>(q_idx); a.q_prob = const_cast<float*>(q_prob); a.q_count = const_cast<int*>(q_count);
    a.R = rows; a.K = k; a.prob_type = prob_type;
    a.buf = (unsigned char*)buf; a.capacity = capacity_bytes; a.bytes_out = bytes_out;
    return wire_common(ctx, a, true, cuda_stream);
}

int picospec_wire_unpack(picospec_ctx* ctx, const void* buf, long long bytes, int rows, int k, int* q_idx,
                         float* q_prob, int* q_count, void* cuda_stream) {
    WireArgs a;
    a.q_idx = q_idx; a.q_prob = q_prob; a.q_count = q_count;
    a.R = rows; a.K = k; a.prob_type = 0;
    a.buf = (unsigned char*)const_cast<void*>(buf); a.capacity = bytes; a.bytes_out = nullptr;
    return wire_common(ctx, a, false, cuda_stream);
}

int picospec_compress(picospec_ctx* ctx, const void* draft_logits, picospec_dtype dtype, int B, int G, int V,
                      long long row_stride_elems, const float* temperature, int top_k, float top_p, int k_max,
                      int* q_idx, float* q_prob, int* q_count, const float* u_draft, int* draft_tok,
                      void* cuda_stream) {
    int rc = check_common(ctx, draft_logits, (int)dtype, B, G, V, row_stride_elems, temperature, k_max);
    if (rc != PICOSPEC_OK) return rc;
    if (!q_idx || !q_prob || !q_count || top_k < 0 || !(top_p > 0.0f)) return PICOSPEC_EINVAL;
    if ((u_draft == nullptr) != (draft_tok == nullptr)) return PICOSPEC_EINVAL;
    if (B == 0 || G == 0) return PICOSPEC_OK;
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail_cuda(ctx, cudaErrorInvalidDevice);
    CompressArgs a;
    a.logits = draft_logits; a.row_stride = row_stride_elems;
    a.B = B; a.G = G; a.V = V; a.nch = (V + CHUNK - 1) / CHUNK; a.k_max = k_max; a.top_k = top_k; a.top_p = top_p;
    a.temperature = temperature; a.q_idx = q_idx; a.q_prob = q_prob; a.q_count = q_count;
    a.u_draft = u_draft; a.draft_tok = draft_tok;
    a.row_pos = nullptr; a.seq_rows = 0; a.raw_probs = 0;
    fill_compress_workspace(ctx, a);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t e;
    if (dtype == PICOSPEC_BF16)
        e = launch_compress<__nv_bfloat16>(ctx, a, rows_aligned(draft_logits, row_stride_elems, 2), s);
    else
        e = launch_compress<float>(ctx, a, rows_aligned(draft_logits, row_stride_elems, 4), s);
    return e == cudaSuccess ? PICOSPEC_OK : fail_cuda(ctx, e);
}

static int verify_common(picospec_ctx* ctx, VerifyArgs& a, picospec_dtype dtype, void* cuda_stream, bool edge = false) {
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail_cuda(ctx, cudaErrorInvalidDevice);
    a.nch = (a.V + CHUNK - 1) / CHUNK;
    if (a.r1 < 0) a.r1 = a.G + 1;
    a.stats = ctx->stats; a.row_max = ctx->row_max; a.dsum = ctx->dsum; a.queue = ctx->queue;
    a.need_rows = ctx->need_rows; a.rowq = ctx->rowq; a.rowq_count = ctx->counters + 5;
    a.queue_count = ctx->counters; a.status = ctx->status; a.slow_rows = ctx->slow_rows;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t e;
    if (dtype == PICOSPEC_BF16)
        e = launch_verify<__nv_bfloat16>(ctx, a, rows_aligned(a.logits, a.row_stride, 2), s, edge);
    else
        e = launch_verify<float>(ctx, a, rows_aligned(a.logits, a.row_stride, 4), s, edge);
    return e == cudaSuccess ? PICOSPEC_OK : fail_cuda(ctx, e);
}

int picospec_verify(picospec_ctx* ctx, const void* target_logits, picospec_dtype dtype, int B, int G, int V,
                    long long row_stride_elems, const float* temperature, const int* draft_tok, const int* q_idx,
                    const float* q_prob, const int* q_count, int k_max, const float* u_accept, int* accept_len,
                    float* p_draft, float* resid_mass, int* borderline_count, const float* u_resample,
                    int* token, void* cuda_stream) {
    int rc = check_common(ctx, target_logits, (int)dtype, B, G, V, row_stride_elems, temperature, k_max);
    if (rc != PICOSPEC_OK) return rc;
    if (!accept_len || !borderline_count) return PICOSPEC_EINVAL;
    if (G > 0 && (!draft_tok || !q_idx || !q_prob || !q_count || !u_accept || !p_draft || !resid_mass))
        return PICOSPEC_EINVAL;
    if ((u_resample == nullptr) != (token == nullptr)) return PICOSPEC_EINVAL;
    if (B == 0) return PICOSPEC_OK;
    VerifyArgs a;
    a.logits = target_logits; a.row_stride = row_stride_elems;
    a.B = B; a.G = G; a.V = V; a.k_max = k_max; a.sample_only = 0;
    a.temperature = temperature; a.draft_tok = draft_tok; a.q_idx = q_idx; a.q_prob = q_prob; a.q_count = q_count;
    a.u_accept = u_accept; a.pos = nullptr; a.u_resample = u_resample;
    a.accept_len = accept_len; a.p_draft = p_draft; a.resid_mass = resid_mass; a.borderline = borderline_count;
    a.token = token; a.mass = nullptr;
    return verify_common(ctx, a, dtype, cuda_stream);
}

int picospec_verify_range(picospec_ctx* ctx, const void* target_logits, picospec_dtype dtype, int B, int G, int V,
                          long long row_stride_elems, const float* temperature, const int* gamma, int r0, int r1,
                          const int* state_in, const int* draft_tok, const int* q_idx, const float* q_prob,
                          const int* q_count, int k_max, const float* u_accept, int* accept_len, float* p_draft,
                          float* resid_mass, int* borderline_count, const float* u_resample, int* token,
                          int* state_out, void* cuda_stream) {
    int rc = check_common(ctx, target_logits, (int)dtype, B, G, V, row_stride_elems, temperature, k_max);
    if (rc != PICOSPEC_OK) return rc;
    if (!accept_len || !borderline_count || !state_out) return PICOSPEC_EINVAL;
    if (r0 < 0 || r1 <= r0 || r1 > G + 1) return PICOSPEC_EINVAL;
    if (G > 0 && (!draft_tok || !q_idx || !q_prob || !q_count || !u_accept || !p_draft || !resid_mass))
        return PICOSPEC_EINVAL;
    if ((u_resample == nullptr) != (token == nullptr)) return PICOSPEC_EINVAL;
    if (B == 0) return PICOSPEC_OK;
    VerifyArgs a;
    a.logits = target_logits; a.row_stride = row_stride_elems;
    a.B = B; a.G = G; a.V = V; a.k_max = k_max; a.sample_only = 0;
    a.r0 = r0; a.r1 = r1; a.gamma = gamma; a.state_in = state_in; a.state_out = state_out;
    a.temperature = temperature; a.draft_tok = draft_tok; a.q_idx = q_idx; a.q_prob = q_prob; a.q_count = q_count;
    a.u_accept = u_accept; a.pos = nullptr; a.u_resample = u_resample;
    a.accept_len = accept_len; a.p_draft = p_draft; a.resid_mass = resid_mass; a.borderline = borderline_count;
    a.token = token; a.mass = nullptr;
    return verify_common(ctx, a, dtype, cuda_stream);
}

int picospec_residual_sample(picospec_ctx* ctx, const void* target_logits, picospec_dtype dtype, int B, int G,
                             int V, long long row_stride_elems, const float* temperature, const int* pos,
                             const int* q_idx, const float* q_prob, const int* q_count, int k_max,
                             const float* u_resample, int* token, float* mass, void* cuda_stream) {
    int rc = check_common(ctx, target_logits, (int)dtype, B, G, V, row_stride_elems, temperature, k_max);
    if (rc != PICOSPEC_OK) return rc;
    if (!pos || !u_resample || !token) return PICOSPEC_EINVAL;
    if (G > 0 && (!q_idx || !q_prob || !q_count)) return PICOSPEC_EINVAL;
    if (B == 0) return PICOSPEC_OK;
    VerifyArgs a;
    a.logits = target_logits; a.row_stride = row_stride_elems;
    a.B = B; a.G = G; a.V = V; a.k_max = k_max; a.sample_only = 1;
    a.temperature = temperature; a.draft_tok = nullptr; a.q_idx = q_idx; a.q_prob = q_prob; a.q_count = q_count;
    a.u_accept = nullptr; a.pos = pos; a.u_resample = u_resample;
    a.accept_len = nullptr; a.p_draft = nullptr; a.resid_mass = nullptr; a.borderline = nullptr;
    a.token = token; a.mass = mass;
    return verify_common(ctx, a, dtype, cuda_stream);
}

int picospec_target_topk(picospec_ctx* ctx, const void* target_logits, picospec_dtype dtype, int B, int R, int V,
                         long long row_stride_elems, const float* temperature, const int* pos, int k, int* p_idx,
                         float* p_prob, int* p_count, void* cuda_stream) {
    int rc = check_common(ctx, target_logits, (int)dtype, B, R > 0 ? R - 1 : -1, V, row_stride_elems, temperature, k);
    if (rc != PICOSPEC_OK) return rc;
    if (!pos || !p_idx || !p_prob || !p_count) return PICOSPEC_EINVAL;
    if (B == 0) return PICOSPEC_OK;
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail_cuda(ctx, cudaErrorInvalidDevice);
    CompressArgs a;
    a.logits = target_logits; a.row_stride = row_stride_elems;
    a.B = B; a.G = 1; a.V = V; a.nch = (V + CHUNK - 1) / CHUNK; a.k_max = k; a.top_k = k; a.top_p = 1.0f;
    a.temperature = temperature; a.q_idx = p_idx; a.q_prob = p_prob; a.q_count = p_count;
    a.u_draft = nullptr; a.draft_tok = nullptr;
    a.row_pos = pos; a.seq_rows = R; a.raw_probs = 1;
    fill_compress_workspace(ctx, a);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t e;
    if (dtype == PICOSPEC_BF16)
        e = launch_compress<__nv_bfloat16>(ctx, a, rows_aligned(target_logits, row_stride_elems, 2), s);
    else
        e = launch_compress<float>(ctx, a, rows_aligned(target_logits, row_stride_elems, 4), s);
    return e == cudaSuccess ? PICOSPEC_OK : fail_cuda(ctx, e);
}

int picospec_edge_resample(picospec_ctx* ctx, const void* draft_logits, picospec_dtype dtype, int B, int R, int V,
                           long long row_stride_elems, const float* temperature, const int* pos, const int* p_idx,
                           const float* p_prob, const int* p_count, int k, const float* u, int* token, float* mass,
                           void* cuda_stream) {
    int rc = check_common(ctx, draft_logits, (int)dtype, B, R > 0 ? R - 1 : -1, V, row_stride_elems, temperature, k);
    if (rc != PICOSPEC_OK) return rc;
    if (!pos || !p_idx || !p_prob || !p_count || !u || !token) return PICOSPEC_EINVAL;
    if (B == 0) return PICOSPEC_OK;
    VerifyArgs a;
    a.logits = draft_logits; a.row_stride = row_stride_elems;
    a.B = B; a.G = R - 1; a.V = V; a.k_max = k; a.sample_only = 1;
    a.temperature = temperature; a.draft_tok = nullptr; a.q_idx = p_idx; a.q_prob = p_prob; a.q_count = p_count;
    a.u_accept = nullptr; a.pos = pos; a.u_resample = u;
    a.accept_len = nullptr; a.p_draft = nullptr; a.resid_mass = nullptr; a.borderline = nullptr;
    a.token = token; a.mass = mass;
    return verify_common(ctx, a, dtype, cuda_stream, true);
}

// ---- vocabulary-parallel verification ---------------------------------------------------------

static int vp_check(const picospec_ctx* ctx, int B, int G, int V, int k_max, int ranks, int chunks_per_rank) {
    if (!ctx) return PICOSPEC_EINVAL;
    if (B < 0 || G < 0 || V <= 0 || k_max <= 0 || ranks < 1 || chunks_per_rank < 1) return PICOSPEC_EINVAL;
    const long long nch = ((long long)V + CHUNK - 1) / CHUNK;
    if ((long long)(ranks - 1) * chunks_per_rank >= nch || (long long)ranks * chunks_per_rank < nch) return PICOSPEC_EINVAL;
    if (B > ctx->max_batch || G > ctx->max_gamma || V > ctx->max_vocab || k_max > ctx->max_k) return PICOSPEC_ECAPACITY;
    return PICOSPEC_OK;
}

// the fields every vocabulary-parallel launch shares
static void vp_args(picospec_ctx* ctx, VerifyArgs& a, int B, int G, int V, int k_max, int chunks_per_rank) {
    a.B = B; a.G = G; a.V = V; a.k_max = k_max; a.sample_only = 0;
    a.nch = (V + CHUNK - 1) / CHUNK;
    a.r0 = 0; a.r1 = G + 1;
    a.chunks_per_rank = chunks_per_rank;
    a.rank_stride = (long long)B * (G + 1) * chunks_per_rank;
    a.row_max = ctx->row_max; a.queue = ctx->queue; a.need_rows = ctx->need_rows;
    a.rowq = ctx->rowq; a.rowq_count = ctx->counters + 5;
    a.queue_count = ctx->counters; a.status = ctx->status; a.slow_rows = ctx->slow_rows;
    a.pos = nullptr; a.mass = nullptr; a.token = nullptr;
    a.draft_tok = nullptr; a.q_idx = nullptr; a.q_prob = nullptr; a.q_count = nullptr;
    a.u_accept = nullptr; a.u_resample = nullptr; a.accept_len = nullptr; a.p_draft = nullptr;
    a.resid_mass = nullptr; a.borderline = nullptr; a.temperature = nullptr;
    a.logits = nullptr; a.row_stride = 0; a.stats = nullptr; a.dsum = nullptr;
}

int picospec_vp_local(picospec_ctx* ctx, const void* slice_logits, picospec_dtype dtype, int B, int G, int Vs, int v0,
                      long long row_stride_elems, int chunks_per_rank, const float* temperature, const int* draft_tok,
                      const int* q_idx, const int* q_count, int k_max, float* records_local, float* entries_local,
                      void* cuda_stream) {
    if (!ctx || !slice_logits || !temperature || !records_local) return PICOSPEC_EINVAL;
    if (dtype != PICOSPEC_F32 && dtype != PICOSPEC_BF16) return PICOSPEC_EINVAL;
    if (B < 0 || G < 0 || Vs <= 0 || v0 < 0 || v0 % CHUNK != 0 || k_max <= 0 || row_stride_elems < Vs) return PICOSPEC_EINVAL;
    const int slice_chunks = (Vs + CHUNK - 1) / CHUNK;
    if (chunks_per_rank < slice_chunks) return PICOSPEC_EINVAL;
    if (G > 0 && (!draft_tok || !q_idx || !q_count || !entries_local)) return PICOSPEC_EINVAL;
    if (B > ctx->max_batch || G > ctx->max_gamma || (long long)v0 + Vs > ctx->max_vocab || k_max > ctx->max_k)
        return PICOSPEC_ECAPACITY;
    if (B == 0) return PICOSPEC_OK;
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail_cuda(ctx, cudaErrorInvalidDevice);
    VerifyArgs a;
    vp_args(ctx, a, B, G, Vs, k_max, 0);
    a.rank_stride = 0;
    a.logits = slice_logits; a.row_stride = row_stride_elems; a.temperature = temperature;
    a.draft_tok = draft_tok; a.q_idx = q_idx; a.q_count = q_count;
    a.stats = reinterpret_cast<float2*>(records_local);
    a.stats_pitch = chunks_per_rank;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t e;
    if (dtype == PICOSPEC_BF16) {
        e = launch_verify_stream<__nv_bfloat16>(ctx, a, rows_aligned(slice_logits, row_stride_elems, 2), s);
        if (e == cudaSuccess && G > 0)
            launch_chained(vp_gather_kernel<__nv_bfloat16>, ctx->num_sms * 4, THREADS, 0, s, a, v0, Vs, entries_local);
    } else {
        e = launch_verify_stream<float>(ctx, a, rows_aligned(slice_logits, row_stride_elems, 4), s);
        if (e == cudaSuccess && G > 0)
            launch_chained(vp_gather_kernel<float>, ctx->num_sms * 4, THREADS, 0, s, a, v0, Vs, entries_local);
    }
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? PICOSPEC_OK : fail_cuda(ctx, e);
}

int picospec_vp_decide(picospec_ctx* ctx, int B, int G, int V, int ranks, int chunks_per_rank, const float* records_all,
                       const double* sums_all, const float* entries_all, const float* temperature, const int* draft_tok,
                       const int* q_idx, const float* q_prob, const int* q_count, int k_max, const float* u_accept,
                       const float* u_resample, int* accept_len, float* p_draft, float* resid_mass,
                       int* borderline_count, int* pick, void* cuda_stream) {
    int rc = vp_check(ctx, B, G, V, k_max, ranks, chunks_per_rank);
    if (rc != PICOSPEC_OK) return rc;
    if (!records_all || !temperature || !accept_len || !borderline_count || !pick || !u_resample) return PICOSPEC_EINVAL;
    if (G > 0 && (!entries_all || !draft_tok || !q_idx || !q_prob || !q_count || !u_accept || !p_draft || !resid_mass))
        return PICOSPEC_EINVAL;
    if (B == 0) return PICOSPEC_OK;
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail_cuda(ctx, cudaErrorInvalidDevice);
    VerifyArgs a;
    vp_args(ctx, a, B, G, V, k_max, chunks_per_rank);
    a.temperature = temperature; a.draft_tok = draft_tok; a.q_idx = q_idx; a.q_prob = q_prob; a.q_count = q_count;
    a.u_accept = u_accept; a.u_resample = u_resample;
    a.accept_len = accept_len; a.p_draft = p_draft; a.resid_mass = resid_mass; a.borderline = borderline_count;
    a.stats = reinterpret_cast<float2*>(const_cast<float*>(records_all));
    a.dsum = const_cast<double*>(sums_all);
    a.entry_logits = entries_all; a.pick = pick;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const size_t dyn = (size_t)a.nch * sizeof(double);
    cudaError_t e = cudaSuccess;
    if (!sums_all) {
        e = cudaMemsetAsync(borderline_count, 0, sizeof(int), s);
        if (e == cudaSuccess) launch_chained(verify_finish_kernel<float, false, true>, B, THREADS, dyn, s, a);
    } else {
        const int g2 = B < ctx->num_sms ? B : ctx->num_sms;
        launch_chained(verify_finish_kernel<float, true, true>, g2, THREADS, dyn, s, a);
    }
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? PICOSPEC_OK : fail_cuda(ctx, e);
}

int picospec_vp_draw(picospec_ctx* ctx, const void* slice_logits, picospec_dtype dtype, int B, int G, int V, int v0,
                     long long row_stride_elems, int rank, int ranks, int chunks_per_rank, const float* records_all,
                     const double* sums_all, const float* temperature, const int* q_idx, const float* q_prob,
                     const int* q_count, int k_max, const float* u_resample, const int* pick, int* tok_flag_local,
                     void* cuda_stream) {
    int rc = vp_check(ctx, B, G, V, k_max, ranks, chunks_per_rank);
    if (rc != PICOSPEC_OK) return rc;
    if (!slice_logits || !records_all || !temperature || !u_resample || !pick || !tok_flag_local) return PICOSPEC_EINVAL;
    if (dtype != PICOSPEC_F32 && dtype != PICOSPEC_BF16) return PICOSPEC_EINVAL;
    if (rank < 0 || rank >= ranks || v0 != rank * chunks_per_rank * CHUNK) return PICOSPEC_EINVAL;
    if (G > 0 && (!q_idx || !q_prob || !q_count)) return PICOSPEC_EINVAL;
    if (B == 0) return PICOSPEC_OK;
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail_cuda(ctx, cudaErrorInvalidDevice);
    VerifyArgs a;
    vp_args(ctx, a, B, G, V, k_max, chunks_per_rank);
    a.logits = slice_logits; a.row_stride = row_stride_elems; a.temperature = temperature;
    a.q_idx = q_idx; a.q_prob = q_prob; a.q_count = q_count; a.u_resample = u_resample;
    a.stats = reinterpret_cast<float2*>(const_cast<float*>(records_all));
    a.dsum = const_cast<double*>(sums_all);
    a.pick = const_cast<int*>(pick);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (dtype == PICOSPEC_BF16) {
        if (sums_all) launch_chained(vp_draw_kernel<__nv_bfloat16, true>, B, THREADS, 0, s, a, v0, rank, ctx->vp_listed, tok_flag_local);
        else launch_chained(vp_draw_kernel<__nv_bfloat16, false>, B, THREADS, 0, s, a, v0, rank, ctx->vp_listed, tok_flag_local);
    } else {
        if (sums_all) launch_chained(vp_draw_kernel<float, true>, B, THREADS, 0, s, a, v0, rank, ctx->vp_listed, tok_flag_local);
        else launch_chained(vp_draw_kernel<float, false>, B, THREADS, 0, s, a, v0, rank, ctx->vp_listed, tok_flag_local);
    }
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? PICOSPEC_OK : fail_cuda(ctx, e);
}

int picospec_vp_queue(picospec_ctx* ctx, int B, int G, const int* pick, const int* tok_flag_all, int* token,
                      void* cuda_stream) {
    if (!ctx || B < 0 || G < 0 || !pick || !tok_flag_all || !token) return PICOSPEC_EINVAL;
    if (B > ctx->max_batch || G > ctx->max_gamma) return PICOSPEC_ECAPACITY;
    if (B == 0) return PICOSPEC_OK;
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail_cuda(ctx, cudaErrorInvalidDevice);
    VerifyArgs a;
    vp_args(ctx, a, B, G, 1, 1, 1);
    a.pick = const_cast<int*>(pick);
    a.token = token;
    launch_chained(vp_queue_kernel, 1, THREADS, 0, (cudaStream_t)cuda_stream, a, tok_flag_all, ctx->vp_listed);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? PICOSPEC_OK : fail_cuda(ctx, e);
}

int picospec_vp_exact(picospec_ctx* ctx, const void* slice_logits, picospec_dtype dtype, int B, int G, int Vs,
                      long long row_stride_elems, int chunks_per_rank, const float* temperature, double* sums_local,
                      void* cuda_stream) {
    if (!ctx || !slice_logits || !temperature || !sums_local) return PICOSPEC_EINVAL;
    if (dtype != PICOSPEC_F32 && dtype != PICOSPEC_BF16) return PICOSPEC_EINVAL;
    if (B < 0 || G < 0 || Vs <= 0 || row_stride_elems < Vs || chunks_per_rank < (Vs + CHUNK - 1) / CHUNK) return PICOSPEC_EINVAL;
    if (B > ctx->max_batch || G > ctx->max_gamma) return PICOSPEC_ECAPACITY;
    if (B == 0) return PICOSPEC_OK;
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail_cuda(ctx, cudaErrorInvalidDevice);
    PreciseArgs p;
    p.logits = slice_logits; p.row_stride = row_stride_elems; p.V = Vs; p.nch = (Vs + CHUNK - 1) / CHUNK;
    p.seq_rows = G + 1; p.temperature = temperature;
    p.rows = ctx->rowq; p.row_count = ctx->counters + 5;
    p.row_max = ctx->row_max; p.dsum = sums_local; p.pitch = chunks_per_rank;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (dtype == PICOSPEC_BF16) launch_chained(precise_chunk_sums_kernel<__nv_bfloat16>, ctx->num_sms * 6, THREADS, 0, s, p);
    else launch_chained(precise_chunk_sums_kernel<float>, ctx->num_sms * 6, THREADS, 0, s, p);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? PICOSPEC_OK : fail_cuda(ctx, e);
}

int picospec_vp_merge(picospec_ctx* ctx, int B, const int* tok_flag_all, int* token, void* cuda_stream) {
    if (!ctx || B < 0 || !tok_flag_all || !token) return PICOSPEC_EINVAL;
    if (B > ctx->max_batch) return PICOSPEC_ECAPACITY;
    if (B == 0) return PICOSPEC_OK;
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail_cuda(ctx, cudaErrorInvalidDevice);
    launch_chained(vp_merge_kernel, (B + THREADS - 1) / THREADS, THREADS, 0, (cudaStream_t)cuda_stream, B, ctx->vp_listed,
                   tok_flag_all, token);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? PICOSPEC_OK : fail_cuda(ctx, e);
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// picospec_verify_static: the verify kernels on a workspace that is part of the device image.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int STATIC_ROWS = PICOSPEC_STATIC_MAX_ROWS;
constexpr int STATIC_NCH = (PICOSPEC_STATIC_MAX_VOCAB + CHUNK - 1) / CHUNK;

struct StaticWorkspace {
    float2 stats[STATIC_ROWS * STATIC_NCH];
    double dsum[STATIC_ROWS * STATIC_NCH];
    float row_max[STATIC_ROWS];
    int queue[STATIC_ROWS];
    int rowq[STATIC_ROWS];
    unsigned long long need_rows[STATIC_ROWS];
    // the words below must read zero when a call starts; one memset covers them
    int counters[4];
    unsigned status;
    unsigned pad;
    unsigned long long slow_rows;
};

// In host code this name is only a handle for cudaGetSymbolAddress, never an address a kernel
// could use; the per-device address is looked up below.
static __device__ __align__(256) unsigned char g_static_workspace[sizeof(StaticWorkspace)];

constexpr int STATIC_MAX_DEVICES = 64;
std::mutex g_static_mutex;
StaticWorkspace* g_static_ptr[STATIC_MAX_DEVICES];   // device address of the array, per device
int g_static_sms[STATIC_MAX_DEVICES];

// Once per device, with that device current: the device address of the array and the SM count.
cudaError_t static_workspace(int device, StaticWorkspace** ws, int* sms) {
    if (device < 0 || device >= STATIC_MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_workspace);
        if (e != cudaSuccess) return e;
        int n = 0;
        e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess) return e;
        g_static_sms[device] = n;
        g_static_ptr[device] = static_cast<StaticWorkspace*>(p);
    }
    *ws = g_static_ptr[device];
    *sms = g_static_sms[device];
    return cudaSuccess;
}

}  // namespace

extern "C" int picospec_verify_static(const void* target_logits, picospec_dtype dtype, int B, int G, int V,
                                      long long row_stride_elems, const float* temperature, const int* draft_tok,
                                      const int* q_idx, const float* q_prob, const int* q_count, int k_max,
                                      const float* u_accept, int* accept_len, float* p_draft, float* resid_mass,
                                      int* borderline_count, const float* u_resample, int* token,
                                      int* device_status_out, long long* slow_rows_out, void* cuda_stream) {
    if (!target_logits || !temperature) return PICOSPEC_EINVAL;
    if (dtype != PICOSPEC_F32 && dtype != PICOSPEC_BF16) return PICOSPEC_EINVAL;
    if (B < 0 || G < 0 || V <= 0 || k_max <= 0 || row_stride_elems < V) return PICOSPEC_EINVAL;
    if (!accept_len || !borderline_count) return PICOSPEC_EINVAL;
    if (G > 0 && (!draft_tok || !q_idx || !q_prob || !q_count || !u_accept || !p_draft || !resid_mass))
        return PICOSPEC_EINVAL;
    if ((u_resample == nullptr) != (token == nullptr)) return PICOSPEC_EINVAL;
    if (G > PICOSPEC_MAX_GAMMA || k_max > PICOSPEC_MAX_K || V > PICOSPEC_STATIC_MAX_VOCAB ||
        (long long)B * (G + 1) > STATIC_ROWS)
        return PICOSPEC_ECAPACITY;
    if (B == 0) return PICOSPEC_OK;

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return PICOSPEC_ECUDA;
    StaticWorkspace* ws = nullptr;
    picospec_ctx local = {};          // host-side launch parameters only; owns nothing
    local.device = device;
    local.wait_limit_ns = WAIT_LIMIT_NS;
    if (static_workspace(device, &ws, &local.num_sms) != cudaSuccess) return PICOSPEC_ECUDA;

    cudaStream_t s = (cudaStream_t)cuda_stream;
    const size_t tail = sizeof(StaticWorkspace) - offsetof(StaticWorkspace, counters);
    if (cudaMemsetAsync(ws->counters, 0, tail, s) != cudaSuccess) return PICOSPEC_ECUDA;

    VerifyArgs a;
    a.logits = target_logits; a.row_stride = row_stride_elems;
    a.B = B; a.G = G; a.V = V; a.k_max = k_max; a.sample_only = 0;
    a.nch = (V + CHUNK - 1) / CHUNK;
    a.r1 = G + 1;
    a.temperature = temperature; a.draft_tok = draft_tok; a.q_idx = q_idx; a.q_prob = q_prob; a.q_count = q_count;
    a.u_accept = u_accept; a.pos = nullptr; a.u_resample = u_resample;
    a.accept_len = accept_len; a.p_draft = p_draft; a.resid_mass = resid_mass; a.borderline = borderline_count;
    a.token = token; a.mass = nullptr;
    a.stats = ws->stats; a.row_max = ws->row_max; a.dsum = ws->dsum; a.queue = ws->queue;
    a.need_rows = ws->need_rows; a.rowq = ws->rowq; a.rowq_count = ws->counters + 1;
    a.queue_count = ws->counters; a.status = &ws->status; a.slow_rows = &ws->slow_rows;
    cudaError_t e;
    if (dtype == PICOSPEC_BF16)
        e = launch_verify<__nv_bfloat16>(&local, a, rows_aligned(a.logits, a.row_stride, 2), s);
    else
        e = launch_verify<float>(&local, a, rows_aligned(a.logits, a.row_stride, 4), s);
    if (e == cudaSuccess && device_status_out)
        e = cudaMemcpyAsync(device_status_out, &ws->status, sizeof(int), cudaMemcpyDeviceToDevice, s);
    if (e == cudaSuccess && slow_rows_out)
        e = cudaMemcpyAsync(slow_rows_out, &ws->slow_rows, sizeof(long long), cudaMemcpyDeviceToDevice, s);
    return e == cudaSuccess ? PICOSPEC_OK : PICOSPEC_ECUDA;
}
