// C ABI of the POP library: argument checking, partition life cycle, stage sequencing.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <vector>

#include "pop_common.cuh"

static thread_local char g_cuda_err[256] = "";

void pop_set_cuda_error(cudaError_t e, const char* what) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s (%s)", what, cudaGetErrorName(e), cudaGetErrorString(e));
    (void)cudaGetLastError();   // clear the sticky-free error state
}

static unsigned long long g_launches = 0;
void pop_count_launch(int n) { __atomic_fetch_add(&g_launches, (unsigned long long)n, __ATOMIC_RELAXED); }
extern "C" unsigned long long pop_kernel_launch_count(void) { return __atomic_load_n(&g_launches, __ATOMIC_RELAXED); }

extern "C" const char* pop_version(void) { return "pop-b200 0.1.0 (sm_100a)"; }

extern "C" const char* pop_last_cuda_error(void) { return g_cuda_err; }

extern "C" const char* pop_status_string(int s) {
    switch (s) {
        case POP_OK: return "POP_OK";
        case POP_ERR_INVALID_ARG: return "POP_ERR_INVALID_ARG";
        case POP_ERR_UNSUPPORTED: return "POP_ERR_UNSUPPORTED";
        case POP_ERR_ALLOC: return "POP_ERR_ALLOC";
        case POP_ERR_CUDA: return "POP_ERR_CUDA";
        case POP_ERR_TIMEOUT: return "POP_ERR_TIMEOUT";
        default: return "POP_ERR_UNKNOWN";
    }
}

extern "C" int pop_region_sizes(int N, pop_ratios_t r, int* n_ret, int* n_cand, int* n_pruned, int* k_default) {
    if (N <= 0) return POP_ERR_INVALID_ARG;
    if (!(r.retained >= 0.0) || !(r.candidate >= 0.0) || !(r.pruned >= 0.0)) return POP_ERR_INVALID_ARG;
    if (r.retained + r.candidate + r.pruned > 1.0 + 1e-9 || r.candidate + r.pruned > 1.0 + 1e-9)
        return POP_ERR_INVALID_ARG;
    const int np = (int)floor(r.pruned * (double)N + 1e-9);
    const int nc = (int)floor(r.candidate * (double)N + 1e-9);
    const int nr = N - np - nc;
    if (nr < 0) return POP_ERR_INVALID_ARG;
    if (n_ret) *n_ret = nr;
    if (n_cand) *n_cand = nc;
    if (n_pruned) *n_pruned = np;
    if (k_default) *k_default = nc / 2;
    return POP_OK;
}

// Device attributes are looked up once per device (the queries are not free on the prefill path).
namespace {
struct DeviceInfo { int valid, sm_count, coop, max_smem_optin; };
const DeviceInfo& device_info(int device) {
    static DeviceInfo info[64];
    static std::mutex m;
    static DeviceInfo fallback;
    DeviceInfo* d = (device >= 0 && device < 64) ? &info[device] : &fallback;
    std::lock_guard<std::mutex> lock(m);
    if (!d->valid) {
        cudaDeviceGetAttribute(&d->sm_count, cudaDevAttrMultiProcessorCount, device);
        cudaDeviceGetAttribute(&d->coop, cudaDevAttrCooperativeLaunch, device);
        cudaDeviceGetAttribute(&d->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
        d->valid = (d != &fallback);
    }
    return *d;
}
}  // namespace

// Temporaries of the prefill come from a stream-ordered pool of the library's own, one per device, that keeps its
// memory when the device goes idle: the device's default pool hands everything back to the driver at each
// synchronisation (release threshold 0), and the first allocation after one then costs several hundred microseconds
// of host time during which the GPU has nothing to do.  What the pool holds is the largest set of temporaries in
// flight (a few MB; tens of MB with pop_prefill_partition_with_output); pop_release_cached_memory() trims it.  If the
// pool cannot be created the default pool serves.
namespace {
struct TempPool { int tried; cudaMemPool_t pool; };
TempPool g_temp_pools[64];
std::mutex g_temp_pool_mutex;

cudaMemPool_t temp_pool(int device) {
    if (device < 0 || device >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_temp_pool_mutex);
    TempPool& t = g_temp_pools[device];
    if (!t.tried) {
        t.tried = 1;
        cudaMemPoolProps props;
        memset(&props, 0, sizeof(props));
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = device;
        cudaMemPool_t pool = nullptr;
        if (cudaMemPoolCreate(&pool, &props) == cudaSuccess) {
            unsigned long long keep = ~0ull;
            if (cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep) == cudaSuccess) t.pool = pool;
            else cudaMemPoolDestroy(pool);
        }
        (void)cudaGetLastError();
    }
    return t.pool;
}

cudaError_t temp_alloc(void** ptr, size_t bytes, int device, cudaStream_t st) {
    cudaMemPool_t pool = temp_pool(device);
    return pool ? cudaMallocFromPoolAsync(ptr, bytes, pool, st) : cudaMallocAsync(ptr, bytes, st);
}

void temp_pools_trim() {
    std::lock_guard<std::mutex> lock(g_temp_pool_mutex);
    for (int i = 0; i < 64; ++i)
        if (g_temp_pools[i].pool) cudaMemPoolTrimTo(g_temp_pools[i].pool, 0);
}
}  // namespace

static bool aligned16(const void* p) { return (((uintptr_t)p) & 15u) == 0; }

static int check_shape(int d, int N, pop_dtype_t dt) {
    if (d <= 0 || N <= 0) return POP_ERR_INVALID_ARG;
    if (dt != POP_F32 && dt != POP_BF16) return POP_ERR_UNSUPPORTED;
    const int es = dt == POP_F32 ? 4 : 2;
    if (((size_t)d * es) % 16 != 0) return POP_ERR_UNSUPPORTED;
    if ((size_t)d * es > 65536) return POP_ERR_UNSUPPORTED;
    return POP_OK;
}

// All device buffers of a partition are carved out of one allocation (one cudaMalloc and one cudaFree per
// partition: the calls, not the bytes, are what a prefill pays for), each on a 256-byte boundary.
struct SlabPlan {
    size_t total = 0;
    size_t take(size_t bytes) {
        const size_t at = total;
        total += ((bytes ? bytes : 16) + 255) & ~(size_t)255;
        return at;
    }
};

// Freed slabs are kept for the next partition of the same device and size instead of going back to the driver:
// a serving loop builds one partition per prompt and layer, and cudaMalloc / cudaFree (which synchronises the
// whole device) would otherwise sit in that path.  The cache holds at most pop_config_t.slab_cache_bytes
// (default 1 GiB; 0 turns it off); what does not fit is freed at once, and pop_release_cached_memory() gives
// everything back.  A slab enters the cache only through pop_partition_destroy, whose contract is that the
// caller has synchronised the work that used it.
namespace {
struct CachedSlab { int device; size_t bytes; void* ptr; };
std::mutex g_slab_mutex;
std::vector<CachedSlab> g_slabs;
size_t g_slab_bytes = 0;

std::mutex g_config_mutex;
PopConfig g_config = {POP_DECODE_AUTO, POP_LAUNCH_PDL, 50000u, 1ull << 30};

size_t slab_cache_limit() { return (size_t)pop_config_snapshot().slab_cache_bytes; }

void* slab_take(int device, size_t bytes) {
    std::lock_guard<std::mutex> lock(g_slab_mutex);
    for (size_t i = 0; i < g_slabs.size(); ++i) {
        if (g_slabs[i].device == device && g_slabs[i].bytes == bytes) {
            void* ptr = g_slabs[i].ptr;
            g_slab_bytes -= bytes;
            g_slabs.erase(g_slabs.begin() + (long)i);
            return ptr;
        }
    }
    return nullptr;
}

void slab_flush() {                      // gives everything back to the driver (cudaFree takes a pointer of any device)
    std::lock_guard<std::mutex> lock(g_slab_mutex);
    for (size_t i = 0; i < g_slabs.size(); ++i) cudaFree(g_slabs[i].ptr);
    g_slabs.clear();
    g_slab_bytes = 0;
}

bool slab_keep(int device, size_t bytes, void* ptr) {
    std::lock_guard<std::mutex> lock(g_slab_mutex);
    if (g_slab_bytes + bytes > slab_cache_limit()) return false;
    g_slabs.push_back(CachedSlab{device, bytes, ptr});
    g_slab_bytes += bytes;
    return true;
}
}  // namespace

PopConfig pop_config_snapshot() {
    std::lock_guard<std::mutex> lock(g_config_mutex);
    return g_config;
}

extern "C" int pop_get_config(pop_config_t* out) {
    if (!out) return POP_ERR_INVALID_ARG;
    const PopConfig c = pop_config_snapshot();
    out->decode_kernel = (pop_decode_kernel_t)c.decode_kernel;
    out->launch_mode = (pop_launch_mode_t)c.launch_mode;
    out->wait_budget_us = c.wait_budget_us;
    out->slab_cache_bytes = c.slab_cache_bytes;
    return POP_OK;
}

extern "C" int pop_set_config(const pop_config_t* in) {
    if (!in) return POP_ERR_INVALID_ARG;
    if (in->decode_kernel < POP_DECODE_AUTO || in->decode_kernel > POP_DECODE_SIMPLE) return POP_ERR_INVALID_ARG;
    if (in->launch_mode < POP_LAUNCH_PDL || in->launch_mode > POP_LAUNCH_PLAIN) return POP_ERR_INVALID_ARG;
    {
        std::lock_guard<std::mutex> lock(g_config_mutex);
        g_config.decode_kernel = in->decode_kernel;
        g_config.launch_mode = in->launch_mode;
        g_config.wait_budget_us = in->wait_budget_us;
        g_config.slab_cache_bytes = in->slab_cache_bytes;
    }
    if (in->slab_cache_bytes == 0) slab_flush();
    return POP_OK;
}

extern "C" int pop_release_cached_memory(void) {
    slab_flush();
    temp_pools_trim();
    return POP_OK;
}

static void partition_free(pop_partition* p) {
    if (!p) return;
    if (p->slab && !slab_keep(p->device, p->slab_bytes, p->slab)) cudaFree(p->slab);
    free(p);
}

// Error paths: work of this call may still be queued on the stream, so the slab goes straight back to the driver
// (after the stream has drained) and never into the cache.
static void partition_free_now(pop_partition* p, cudaStream_t st) {
    if (!p) return;
    cudaStreamSynchronize(st);
    if (p->slab) cudaFree(p->slab);
    free(p);
}

// Allocates the partition's buffers for given region sizes (contents undefined except zeroed scratch).
static int partition_alloc(int d, int N, pop_dtype_t dt, int n_ret, int n_cand, cudaStream_t st, pop_partition** out) {
    pop_partition* p = (pop_partition*)calloc(1, sizeof(pop_partition));
    if (!p) return POP_ERR_ALLOC;
    cudaError_t e = cudaGetDevice(&p->device);
    if (e != cudaSuccess) { pop_set_cuda_error(e, "cudaGetDevice"); free(p); return POP_ERR_CUDA; }
    p->d = d; p->N = N; p->dtype = dt; p->es = dt == POP_F32 ? 4 : 2;
    p->n_ret = n_ret; p->n_cand = n_cand; p->n_pruned = N - n_ret - n_cand; p->n_rc = n_ret + n_cand;
    const DeviceInfo& di = device_info(p->device);
    p->sm_count = di.sm_count; p->coop = di.coop; p->max_smem_optin = di.max_smem_optin;
    const size_t row = (size_t)d * p->es;
    // pop_config_t.decode_kernel (as it stands when the partition is created) picks the decode kernel family.
    // POP_DECODE_AUTO: tiled layout + the dataflow kernel of pop_decode_stream.cu for the bf16 shapes it takes (its
    // one-warp selection holds up to pop_stream_max_candidates() = 3072 keys), row layout + the fused / simple kernels for every other
    // shape; POP_DECODE_FUSED / POP_DECODE_SIMPLE: row layout and those kernels for all shapes.
    const int want = pop_config_snapshot().decode_kernel;
    p->layout = (want == POP_DECODE_AUTO && pop_stream_layout_supported(d, dt) && n_cand <= pop_stream_max_candidates()) ? POP_LAYOUT_TILED : POP_LAYOUT_ROWS;
    p->force_simple = want == POP_DECODE_SIMPLE;
    p->n_rt = (n_ret + 7) / 8;
    p->n_cg = (n_ret + 15) / 16;
    p->n_ct = (n_cand + 7) / 8;
    p->n_ret_pad = 16 * p->n_cg;
    p->h_stride = p->layout == POP_LAYOUT_TILED ? p->n_ret_pad + ((n_cand + 15) / 16) * 16 : (p->n_rc > 0 ? p->n_rc : 1);
    SlabPlan plan;
    const size_t o_GU = plan.take(p->layout == POP_LAYOUT_TILED ? ((size_t)(p->n_rt + p->n_ct) * 16 + (size_t)n_cand * 2) * row
                                                                : (size_t)p->n_rc * 2 * row);
    const size_t o_WdT = plan.take(p->layout == POP_LAYOUT_TILED ? ((size_t)p->n_ret_pad + (size_t)n_cand) * row
                                                                 : (size_t)p->n_rc * row);
    const size_t o_ret = plan.take(sizeof(int32_t) * (size_t)n_ret);
    const size_t o_cand = plan.take(sizeof(int32_t) * (size_t)n_cand);
    const size_t o_pruned = plan.take(sizeof(int32_t) * (size_t)p->n_pruned);
    const size_t o_norm = plan.take(sizeof(double) * (size_t)n_cand);
    const size_t o_keys = plan.take(sizeof(u64) * (size_t)n_cand);
    const size_t o_sel = plan.take(sizeof(int32_t) * (size_t)n_cand);
    const size_t o_wnorm = plan.take(sizeof(float) * 2 * (size_t)(n_cand > 0 ? n_cand : 1));
    const size_t o_rpart = plan.take(sizeof(double) * 4 * POP_MAX_BATCH * (size_t)(n_cand > 0 ? n_cand : 1));
    // everything that must start at zero sits in one run, cleared by one memset
    const size_t o_zero = plan.total;
    const size_t o_scores = plan.take(sizeof(double) * (size_t)N);
    const size_t o_bounds = plan.take(sizeof(double) * (size_t)N);
    const size_t o_rank = plan.take(sizeof(int32_t) * (size_t)N);
    // (tiled layout: 8 bytes per element of h, the value with the epoch of the step that wrote it)
    const size_t h_bytes = 2 * sizeof(float) * (size_t)POP_MAX_BATCH * (size_t)(p->h_stride > 0 ? p->h_stride : 1);
    const size_t o_h = plan.take(h_bytes);
    const size_t o_yacc = plan.take(sizeof(float) * (size_t)POP_MAX_BATCH * d);
    const size_t o_sync = plan.take(sizeof(u32) * SYNC_WORDS);
    const size_t zero_bytes = plan.total - o_zero;
    p->slab_bytes = plan.total;
    p->slab = slab_take(p->device, plan.total);
    e = p->slab ? cudaSuccess : cudaMalloc(&p->slab, plan.total);
    if (e == cudaErrorMemoryAllocation) {          // out of memory with slabs in the cache: give them back and try again
        (void)cudaGetLastError();
        slab_flush();
        e = cudaMalloc(&p->slab, plan.total);
    }
    if (e != cudaSuccess) {
        pop_set_cuda_error(e, "cudaMalloc");
        free(p);
        return e == cudaErrorMemoryAllocation ? POP_ERR_ALLOC : POP_ERR_CUDA;
    }
    unsigned char* base = (unsigned char*)p->slab;
    p->GU = base + o_GU; p->WdT = base + o_WdT;
    p->idx_ret = (int32_t*)(base + o_ret); p->idx_cand = (int32_t*)(base + o_cand); p->idx_pruned = (int32_t*)(base + o_pruned);
    p->scores = (double*)(base + o_scores); p->score_bounds = (double*)(base + o_bounds); p->norm_cand = (double*)(base + o_norm);
    p->h = (float*)(base + o_h); p->keys = (u64*)(base + o_keys); p->y_acc = (float*)(base + o_yacc);
    p->sel_slots = (int32_t*)(base + o_sel); p->rank_tmp = (int32_t*)(base + o_rank); p->sync = (u32*)(base + o_sync);
    p->wnorm_cand = (float*)(base + o_wnorm); p->rpart = (double*)(base + o_rpart);
    e = cudaMemsetAsync(base + o_zero, 0, zero_bytes, st);
    if (e != cudaSuccess) { pop_set_cuda_error(e, "cudaMemsetAsync"); partition_free_now(p, st); return POP_ERR_CUDA; }
    *out = p;
    return POP_OK;
}

// Statistics of a weight set into caller-provided device arrays (norm [N]; gnorm, unorm [n_pad] for bf16 with a
// tensor-core prefill, else unused).
static int launch_weight_stats(const void* Wg, const void* Wu, const void* Wd, int N, int d, pop_dtype_t dtype,
                               double* norm, float* gnorm, float* unorm, int n_pad, cudaStream_t st) {
    int rc = pop_launch_colnorm(Wd, d, N, dtype, norm, st);
    if (rc == POP_OK && pop_prefill_tc_supported(d, dtype)) rc = pop_launch_weight_rownorms(Wg, Wu, N, n_pad, d, gnorm, unorm, st);
    return rc;
}

extern "C" int pop_weights_prepare(const void* Wg, const void* Wu, const void* Wd, int N, int d, pop_dtype_t dtype,
                                   void* cuda_stream, pop_weights_t** out) {
    if (!out) return POP_ERR_INVALID_ARG;
    *out = nullptr;
    if (!Wg || !Wu || !Wd) return POP_ERR_INVALID_ARG;
    int rc = check_shape(d, N, dtype);
    if (rc != POP_OK) return rc;
    if (!aligned16(Wg) || !aligned16(Wu) || !aligned16(Wd)) return POP_ERR_INVALID_ARG;
    pop_weights* w = (pop_weights*)calloc(1, sizeof(pop_weights));
    if (!w) return POP_ERR_ALLOC;
    cudaError_t e = cudaGetDevice(&w->device);
    if (e != cudaSuccess) { pop_set_cuda_error(e, "cudaGetDevice"); free(w); return POP_ERR_CUDA; }
    w->d = d; w->N = N; w->dtype = dtype; w->Wg = Wg; w->Wu = Wu; w->Wd = Wd;
    const bool tc = pop_prefill_tc_supported(d, dtype);
    PrefillTcPlan tp;
    pop_prefill_tc_plan(1, d, N, &tp);
    SlabPlan plan;
    const size_t o_norm = plan.take(sizeof(double) * (size_t)N);
    const size_t o_gn = plan.take(tc ? sizeof(float) * (size_t)tp.n_pad : 0);
    const size_t o_un = plan.take(tc ? sizeof(float) * (size_t)tp.n_pad : 0);
    e = cudaMalloc(&w->block, plan.total);
    if (e != cudaSuccess) { pop_set_cuda_error(e, "cudaMalloc"); free(w); return e == cudaErrorMemoryAllocation ? POP_ERR_ALLOC : POP_ERR_CUDA; }
    unsigned char* base = (unsigned char*)w->block;
    w->norm = (double*)(base + o_norm);
    w->gnorm = tc ? (float*)(base + o_gn) : nullptr;
    w->unorm = tc ? (float*)(base + o_un) : nullptr;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    rc = launch_weight_stats(Wg, Wu, Wd, N, d, dtype, w->norm, w->gnorm, w->unorm, tp.n_pad, st);
    if (rc == POP_OK && tc) {
        rc = pop_prefill_tc_encode_weight_maps(Wg, Wu, N, d, w->map_g, w->map_u);
        w->have_maps = rc == POP_OK;
    }
    if (rc != POP_OK) { cudaStreamSynchronize(st); cudaFree(w->block); free(w); return rc; }
    *out = w;
    return POP_OK;
}

extern "C" int pop_weights_destroy(pop_weights_t* w) {
    if (!w) return POP_ERR_INVALID_ARG;
    if (w->block) cudaFree(w->block);
    free(w);
    return POP_OK;
}

// The prefilling stage proper.  `prepared` (may be NULL) carries the statistics of the weight set; without it they
// are computed into this call's temporaries.
static int prefill_partition_impl(const void* X, int L, int d, const void* Wg, const void* Wu, const void* Wd, int N,
                                  pop_dtype_t dtype, pop_ratios_t ratios, const pop_weights* prepared, cudaStream_t st,
                                  pop_partition_t** out, int k_out = -1, void* Y = nullptr, int token_stride = 1) {
    int n_ret, n_cand, n_pruned;
    int rc = pop_region_sizes(N, ratios, &n_ret, &n_cand, &n_pruned, nullptr);
    if (rc != POP_OK) return rc;
    const bool want_y = Y != nullptr;
    if (want_y) {
        if (k_out < 0 || k_out > n_cand) return POP_ERR_INVALID_ARG;
        if (!pop_prefill_output_supported(d, N, dtype)) return POP_ERR_UNSUPPORTED;
    }
    pop_partition* p = nullptr;
    rc = partition_alloc(d, N, dtype, n_ret, n_cand, st, &p);
    if (rc != POP_OK) return rc;

    // temporaries (one stream-ordered allocation, freed in stream order): column norms, activation energies and,
    // for the tensor-core pass, its partial sums, bounds and the re-scoring list
    // partial probing: the statistics come from every token_stride-th prompt token, gathered into a temporary
    const int L_all = L;
    if (token_stride > 1) L = (L + token_stride - 1) / token_stride;
    const bool tc = pop_prefill_tc_supported(d, dtype);
    const bool gemm = pop_prefill_s2_gemm_supported(d);
    PrefillTcPlan tp;
    pop_prefill_tc_plan(L, d, N, &tp);
    SlabPlan tmp;
    const size_t t_probe = tmp.take(token_stride > 1 ? (size_t)L * d * p->es : 0);
    const size_t t_norm = tmp.take(prepared ? 0 : sizeof(double) * (size_t)N);
    const size_t t_s2 = tmp.take(tc ? 0 : sizeof(double) * (size_t)N);
    const size_t t_s2part = tmp.take(gemm ? sizeof(double) * (size_t)N * (size_t)pop_prefill_s2_gemm_splits(L) : 0);
    size_t t_xn = 0, t_gn = 0, t_un = 0, t_tp = 0, t_bp = 0, t_mm = 0, t_list = 0, t_nl = 0, t_part = 0, t_H = 0;
    if (tc) {
        t_H = tmp.take(want_y ? sizeof(__nv_bfloat16) * 2 * (size_t)tp.l_pad * tp.n_pad : 0);
        t_xn = tmp.take(sizeof(float) * (size_t)tp.l_pad);
        t_gn = tmp.take(prepared ? 0 : sizeof(float) * (size_t)tp.n_pad);
        t_un = tmp.take(prepared ? 0 : sizeof(float) * (size_t)tp.n_pad);
        t_tp = tmp.take(sizeof(double) * (size_t)tp.n_parts * tp.n_pad);
        t_bp = tmp.take(sizeof(float) * (size_t)tp.n_parts * tp.n_pad);
        t_mm = tmp.take(sizeof(u64));
        t_list = tmp.take(sizeof(int32_t) * (size_t)N);
        t_nl = tmp.take(sizeof(int));
        t_part = tmp.take(sizeof(double) * (size_t)tp.max_list * tp.n_tb);
    }
    unsigned char* tb = nullptr;
    cudaError_t e = temp_alloc((void**)&tb, tmp.total, p->device, st);
    if (e != cudaSuccess) {
        pop_set_cuda_error(e, "cudaMallocAsync");
        partition_free_now(p, st);
        return POP_ERR_ALLOC;
    }
    if (token_stride > 1) {
        rc = pop_launch_gather_rows(X, L_all, (size_t)d * p->es, token_stride, tb + t_probe, st);
        X = tb + t_probe;
    }
    WeightStats ws;
    if (rc == POP_OK && prepared) {
        ws.norm = prepared->norm; ws.gnorm = prepared->gnorm; ws.unorm = prepared->unorm;
        ws.map_g = prepared->have_maps ? prepared->map_g : nullptr;
        ws.map_u = prepared->have_maps ? prepared->map_u : nullptr;
    } else if (rc == POP_OK) {
        double* norm = (double*)(tb + t_norm);
        float *gn = (float*)(tb + t_gn), *un = (float*)(tb + t_un);
        rc = launch_weight_stats(Wg, Wu, Wd, N, d, dtype, norm, gn, un, tp.n_pad, st);
        ws.norm = norm; ws.gnorm = gn; ws.unorm = un; ws.map_g = nullptr; ws.map_u = nullptr;
    }
    double* s2part = (double*)(tb + t_s2part);
    PrefillTcScratch sc;
    if (rc == POP_OK && tc) {
        sc.xnorm = (float*)(tb + t_xn); sc.gnorm = nullptr; sc.unorm = nullptr;
        sc.H = want_y ? (void*)(tb + t_H) : nullptr;
        sc.s2part = (double*)(tb + t_tp); sc.bpart = (float*)(tb + t_bp); sc.m_max = (u64*)(tb + t_mm);
        sc.list = (int32_t*)(tb + t_list); sc.n_list = (int*)(tb + t_nl); sc.part = (double*)(tb + t_part);
        sc.rank = p->rank_tmp;
        sc.s2part_full = s2part;
        rc = pop_launch_prefill_tc(X, L, d, Wg, Wu, N, ws, sc, p->scores, p->score_bounds, p->sync + SYNC_ERROR, p->sm_count, st);
        if (rc == POP_OK)
            rc = pop_launch_prefill_rescore(X, L, d, Wg, Wu, N, ws.norm, n_ret, n_cand, want_y ? n_ret + k_out : 0, sc, p->scores,
                                            p->score_bounds, p->sm_count, st);
    } else if (rc == POP_OK) {
        double* s2 = (double*)(tb + t_s2);
        rc = gemm ? pop_launch_prefill_s2_gemm(X, L, d, Wg, Wu, N, dtype, s2part, s2, st)
                  : pop_launch_prefill_s2_exact(X, L, d, Wg, Wu, N, dtype, nullptr, N, s2, st);
        // (rank_tmp is still zero from the partition's creation; scores_kernel clears it all the same)
        if (rc == POP_OK) rc = pop_launch_scores(s2, ws.norm, N, p->scores, p->rank_tmp, st);
    }
    if (rc == POP_OK)
        rc = tc ? pop_launch_partition_after_rescore(p->scores, N, n_ret, n_cand, p->rank_tmp, p->sm_count, sc.list, sc.n_list,
                                                     tp.max_list, p->idx_ret, p->idx_cand, p->idx_pruned, st)
                : pop_launch_partition(p->scores, N, n_ret, n_cand, p->rank_tmp, p->sm_count, p->idx_ret, p->idx_cand, p->idx_pruned, st);
    if (rc == POP_OK) rc = p->layout == POP_LAYOUT_TILED ? pop_launch_repack_tiled(p, Wg, Wu, Wd, ws.norm, st)
                                                         : pop_launch_repack(p, Wg, Wu, Wd, ws.norm, st);
    // the prompt's own output under the mask rank < n_ret + k (the ranks are final for every channel near that boundary)
    if (rc == POP_OK && want_y)
        rc = pop_launch_prefill_output(sc.H, L, d, Wd, N, p->rank_tmp, n_ret + k_out, Y, p->sync + SYNC_ERROR, p->sm_count, st);
    cudaFreeAsync(tb, st);
    if (rc != POP_OK) { partition_free_now(p, st); return rc; }
    *out = p;
    return POP_OK;
}

extern "C" int pop_prefill_partition_with_output(const void* X, int L, const pop_weights_t* w, pop_ratios_t ratios,
                                                 int k_candidate, void* Y, void* cuda_stream, pop_partition_t** out) {
    if (!out) return POP_ERR_INVALID_ARG;
    *out = nullptr;
    if (!X || !w || !Y || L <= 0 || !aligned16(X) || !aligned16(Y)) return POP_ERR_INVALID_ARG;
    int dev = -1;
    POP_CUDA(cudaGetDevice(&dev));
    if (dev != w->device) return POP_ERR_INVALID_ARG;
    return prefill_partition_impl(X, L, w->d, w->Wg, w->Wu, w->Wd, w->N, w->dtype, ratios, w, (cudaStream_t)cuda_stream, out,
                                  k_candidate, Y);
}

extern "C" int pop_prefill_partition(const void* X, int L, int d, const void* Wg, const void* Wu, const void* Wd,
                                     int N, pop_dtype_t dtype, pop_ratios_t ratios, void* cuda_stream,
                                     pop_partition_t** out) {
    if (!out) return POP_ERR_INVALID_ARG;
    *out = nullptr;
    if (!X || !Wg || !Wu || !Wd || L <= 0) return POP_ERR_INVALID_ARG;
    int rc = check_shape(d, N, dtype);
    if (rc != POP_OK) return rc;
    if (!aligned16(X) || !aligned16(Wg) || !aligned16(Wu) || !aligned16(Wd)) return POP_ERR_INVALID_ARG;
    return prefill_partition_impl(X, L, d, Wg, Wu, Wd, N, dtype, ratios, nullptr, (cudaStream_t)cuda_stream, out);
}

extern "C" int pop_prefill_partition_prepared(const void* X, int L, const pop_weights_t* w, pop_ratios_t ratios,
                                              void* cuda_stream, pop_partition_t** out) {
    if (!out) return POP_ERR_INVALID_ARG;
    *out = nullptr;
    if (!X || !w || L <= 0 || !aligned16(X)) return POP_ERR_INVALID_ARG;
    int dev = -1;
    POP_CUDA(cudaGetDevice(&dev));
    if (dev != w->device) return POP_ERR_INVALID_ARG;
    return prefill_partition_impl(X, L, w->d, w->Wg, w->Wu, w->Wd, w->N, w->dtype, ratios, w, (cudaStream_t)cuda_stream, out);
}

extern "C" int pop_prefill_partition_probe(const void* X, int L, int token_stride, const pop_weights_t* w, pop_ratios_t ratios,
                                           void* cuda_stream, pop_partition_t** out) {
    if (!out) return POP_ERR_INVALID_ARG;
    *out = nullptr;
    if (!X || !w || L <= 0 || token_stride < 1 || !aligned16(X)) return POP_ERR_INVALID_ARG;
    int dev = -1;
    POP_CUDA(cudaGetDevice(&dev));
    if (dev != w->device) return POP_ERR_INVALID_ARG;
    return prefill_partition_impl(X, L, w->d, w->Wg, w->Wu, w->Wd, w->N, w->dtype, ratios, w, (cudaStream_t)cuda_stream, out,
                                  -1, nullptr, token_stride);
}

extern "C" int pop_partition_from_indices(const void* Wg, const void* Wu, const void* Wd, int N, int d,
                                          pop_dtype_t dtype, const int32_t* h_ret, int n_ret,
                                          const int32_t* h_cand, int n_cand, void* cuda_stream,
                                          pop_partition_t** out) {
    if (!out) return POP_ERR_INVALID_ARG;
    *out = nullptr;
    if (!Wg || !Wu || !Wd || n_ret < 0 || n_cand < 0) return POP_ERR_INVALID_ARG;
    if ((n_ret > 0 && !h_ret) || (n_cand > 0 && !h_cand)) return POP_ERR_INVALID_ARG;
    int rc = check_shape(d, N, dtype);
    if (rc != POP_OK) return rc;
    if (!aligned16(Wg) || !aligned16(Wu) || !aligned16(Wd)) return POP_ERR_INVALID_ARG;
    if ((long long)n_ret + n_cand > N) return POP_ERR_INVALID_ARG;
    // ascending, in range, disjoint
    unsigned char* seen = (unsigned char*)calloc((size_t)N, 1);
    if (!seen) return POP_ERR_ALLOC;
    bool ok = true;
    for (int pass = 0; pass < 2 && ok; ++pass) {
        const int32_t* a = pass ? h_cand : h_ret;
        const int n = pass ? n_cand : n_ret;
        for (int i = 0; i < n; ++i) {
            if (a[i] < 0 || a[i] >= N || (i > 0 && a[i] <= a[i - 1]) || seen[a[i]]) { ok = false; break; }
            seen[a[i]] = 1;
        }
    }
    int32_t* h_pruned = nullptr;
    const int n_pruned = N - n_ret - n_cand;
    if (ok) {
        h_pruned = (int32_t*)malloc(sizeof(int32_t) * (size_t)(n_pruned > 0 ? n_pruned : 1));
        if (h_pruned) { int q = 0; for (int i = 0; i < N; ++i) if (!seen[i]) h_pruned[q++] = i; }
    }
    free(seen);
    if (!ok) return POP_ERR_INVALID_ARG;
    if (!h_pruned) return POP_ERR_ALLOC;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    pop_partition* p = nullptr;
    rc = partition_alloc(d, N, dtype, n_ret, n_cand, st, &p);
    if (rc != POP_OK) { free(h_pruned); return rc; }
    cudaError_t e = cudaSuccess;
    if (n_ret) e = cudaMemcpyAsync(p->idx_ret, h_ret, sizeof(int32_t) * (size_t)n_ret, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && n_cand) e = cudaMemcpyAsync(p->idx_cand, h_cand, sizeof(int32_t) * (size_t)n_cand, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && n_pruned) e = cudaMemcpyAsync(p->idx_pruned, h_pruned, sizeof(int32_t) * (size_t)n_pruned, cudaMemcpyHostToDevice, st);
    // the host arrays are pageable: wait so that the caller (and h_pruned) may go away
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    free(h_pruned);
    if (e != cudaSuccess) { pop_set_cuda_error(e, "index upload"); partition_free_now(p, st); return POP_ERR_CUDA; }
    double* norm = nullptr;
    e = temp_alloc((void**)&norm, sizeof(double) * (size_t)N, p->device, st);
    if (e != cudaSuccess) { pop_set_cuda_error(e, "cudaMallocAsync"); partition_free_now(p, st); return POP_ERR_ALLOC; }
    rc = pop_launch_colnorm(Wd, d, N, dtype, norm, st);
    if (rc == POP_OK) rc = p->layout == POP_LAYOUT_TILED ? pop_launch_repack_tiled(p, Wg, Wu, Wd, norm, st)
                                                         : pop_launch_repack(p, Wg, Wu, Wd, norm, st);
    cudaFreeAsync(norm, st);
    if (rc != POP_OK) { partition_free_now(p, st); return rc; }
    *out = p;
    return POP_OK;
}

extern "C" int pop_partition_sizes(const pop_partition_t* p, int* n_ret, int* n_cand, int* n_pruned) {
    if (!p) return POP_ERR_INVALID_ARG;
    if (n_ret) *n_ret = p->n_ret;
    if (n_cand) *n_cand = p->n_cand;
    if (n_pruned) *n_pruned = p->n_pruned;
    return POP_OK;
}

extern "C" int pop_partition_indices(const pop_partition_t* p, const int32_t** d_ret, const int32_t** d_cand,
                                     const int32_t** d_pruned) {
    if (!p) return POP_ERR_INVALID_ARG;
    if (d_ret) *d_ret = p->idx_ret;
    if (d_cand) *d_cand = p->idx_cand;
    if (d_pruned) *d_pruned = p->idx_pruned;
    return POP_OK;
}

extern "C" int pop_partition_scores(const pop_partition_t* p, const double** d_scores) {
    if (!p || !d_scores) return POP_ERR_INVALID_ARG;
    *d_scores = p->scores;
    return POP_OK;
}

extern "C" int pop_partition_score_bounds(const pop_partition_t* p, const double** d_bounds) {
    if (!p || !d_bounds) return POP_ERR_INVALID_ARG;
    *d_bounds = p->score_bounds;
    return POP_OK;
}

extern "C" int pop_partition_streamed_scores(const pop_partition_t* p, const float** d_score_bound_pairs) {
    if (!p || !d_score_bound_pairs) return POP_ERR_INVALID_ARG;
    if (p->layout != POP_LAYOUT_TILED) return POP_ERR_UNSUPPORTED;
    *d_score_bound_pairs = reinterpret_cast<const float*>(p->keys);
    return POP_OK;
}

extern "C" int pop_partition_shape(const pop_partition_t* p, int* d, int* N, pop_dtype_t* dtype) {
    if (!p) return POP_ERR_INVALID_ARG;
    if (d) *d = p->d;
    if (N) *N = p->N;
    if (dtype) *dtype = p->dtype;
    return POP_OK;
}

extern "C" int pop_partition_check(pop_partition_t* p) {
    if (!p) return POP_ERR_INVALID_ARG;
    POP_CUDA(cudaDeviceSynchronize());
    u32 flag = 0;
    POP_CUDA(cudaMemcpy(&flag, p->sync + SYNC_ERROR, sizeof(u32), cudaMemcpyDeviceToHost));
    if (flag) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "a bounded device-side wait expired in a decode step (wait code %u)", flag);
        // leave the partition usable: clear counters and the accumulator
        POP_CUDA(cudaMemset(p->sync, 0, sizeof(u32) * SYNC_WORDS));
        POP_CUDA(cudaMemset(p->y_acc, 0, sizeof(float) * (size_t)POP_MAX_BATCH * p->d));
        POP_CUDA(cudaMemset(p->h, 0, 2 * sizeof(float) * (size_t)POP_MAX_BATCH * (size_t)(p->h_stride > 0 ? p->h_stride : 1)));
        return POP_ERR_TIMEOUT;
    }
    return POP_OK;
}

extern "C" int pop_partition_destroy(pop_partition_t* p) {
    if (!p) return POP_ERR_INVALID_ARG;
    partition_free(p);
    return POP_OK;
}

extern "C" int pop_decode_step(pop_partition_t* p, const void* x, int B, int k_candidate, void* y,
                               uint8_t* mask_out, int32_t* sel_out, void* cuda_stream) {
    if (!p || !x || !y) return POP_ERR_INVALID_ARG;
    if (B < 1 || k_candidate < 0 || k_candidate > p->n_cand) return POP_ERR_INVALID_ARG;
    if (B > POP_MAX_BATCH) return POP_ERR_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(y)) return POP_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (p->layout == POP_LAYOUT_TILED) return pop_launch_decode_stream(p, x, B, k_candidate, y, mask_out, sel_out, st);
    int rc = pop_launch_decode(p, x, B, k_candidate, y, mask_out, sel_out, st);
    if (rc == POP_ERR_UNSUPPORTED) rc = pop_launch_decode_simple(p, x, B, k_candidate, y, mask_out, sel_out, st);
    return rc;
}
