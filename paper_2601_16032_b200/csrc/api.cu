// C-ABI entry points of libsawtooth_attn: argument validation, launch plan, tensor maps, launch.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "../../include/sawtooth_attn.h"
#include "attn_fwd_sm100.cuh"

namespace {

using namespace sawtooth;

thread_local char g_error[512] = "";

int fail(int status, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof(g_error), fmt, ap);
    va_end(ap);
    return status;
}

__device__ int g_status_word = 0;
__device__ unsigned long long g_cycles = 0;

// Scratch of attn_fwd_dynamic_noalloc: the claim counter block and one counter per CTA, resident in every GPU
// that loads the library for as long as the process lives.
static __device__ __align__(256) int g_noalloc_scratch[(ATTN_DYNAMIC_SCRATCH_HEADER / 4) + ATTN_NOALLOC_MAX_CTAS];
constexpr int kMaxDevices = 64;
int* g_noalloc_ptr[kMaxDevices] = {};  // device address of the array above, per device, once looked up

constexpr int kMaxHostChunks = 16;
constexpr int kSmemOptinB200 = 232448;  // 227 KiB of dynamic shared memory per CTA on sm_100

struct Resolved {
    int block_n, q_tiles, stages, head_fastest, launch_mode, l2_policy, max_ctas;
    size_t smem;
};

size_t smem_for(int d, int block_n, int q_tiles, int stages) {
    return (size_t)q_tiles * kBlockM * d * 2 + (size_t)stages * block_n * d * 2 + sizeof(Barriers);
}

int check_shape(int B, int H, int N, int d, int causal, int dtype) {
    if (B <= 0 || H <= 0 || N <= 0) return fail(ATTN_ERR_INVALID_ARG, "B, H and N must be positive (got %d, %d, %d)", B, H, N);
    if ((long long)B * H > 2147483647LL) return fail(ATTN_ERR_INVALID_ARG, "B*H exceeds 2^31-1");
    if (N > (1 << 24)) return fail(ATTN_ERR_INVALID_ARG, "N exceeds 2^24");
    if (d != 64 && d != 128) return fail(ATTN_ERR_UNSUPPORTED, "head dimension %d is not supported (64 or 128)", d);
    if (causal != 0 && causal != 1) return fail(ATTN_ERR_INVALID_ARG, "causal must be 0 or 1");
    if (dtype != ATTN_F16 && dtype != ATTN_BF16) return fail(ATTN_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    return ATTN_OK;
}

int resolve_opts(const attn_fwd_opts* o, int d, int smem_limit, Resolved* r) {
    attn_fwd_opts z;
    memset(&z, 0, sizeof(z));
    if (o) z = *o;
    r->block_n = z.block_n ? z.block_n : 128;
    r->q_tiles = z.q_tiles ? z.q_tiles : 2;
    if (r->block_n != 64 && r->block_n != 128) return fail(ATTN_ERR_INVALID_ARG, "block_n must be 64 or 128");
    if (r->q_tiles != 1 && r->q_tiles != 2) return fail(ATTN_ERR_INVALID_ARG, "q_tiles must be 1 or 2");
    if (z.digit_order != ATTN_TILE_FASTEST && z.digit_order != ATTN_HEAD_FASTEST)
        return fail(ATTN_ERR_INVALID_ARG, "unknown digit_order %d", z.digit_order);
    if (z.launch_mode != 0 && z.launch_mode != 1) return fail(ATTN_ERR_INVALID_ARG, "launch_mode must be 0 or 1");
    if (z.l2_policy != 0 && z.l2_policy != 1) return fail(ATTN_ERR_INVALID_ARG, "l2_policy must be 0 or 1");
    if (z.max_ctas < 0 || z.kv_stages < 0) return fail(ATTN_ERR_INVALID_ARG, "max_ctas and kv_stages must be >= 0");
    if (z.host_chunks < 0 || z.host_chunks > kMaxHostChunks) return fail(ATTN_ERR_INVALID_ARG, "host_chunks must be in [0, %d]", kMaxHostChunks);
    r->head_fastest = z.digit_order == ATTN_HEAD_FASTEST;
    r->launch_mode = z.launch_mode;
    r->l2_policy = z.l2_policy;
    r->max_ctas = z.max_ctas;
    int fit = 0;
    for (int s = kMaxStages; s >= 2; --s)
        if (smem_for(d, r->block_n, r->q_tiles, s) <= (size_t)smem_limit) { fit = s; break; }
    if (fit == 0) return fail(ATTN_ERR_UNSUPPORTED, "tile configuration does not fit in shared memory");
    if (z.kv_stages) {
        if (z.kv_stages < 2 || z.kv_stages > fit)
            return fail(ATTN_ERR_INVALID_ARG, "kv_stages must be in [2, %d] for this configuration", fit);
        fit = z.kv_stages;
    }
    r->stages = fit;
    r->smem = smem_for(d, r->block_n, r->q_tiles, fit);
    return ATTN_OK;
}

int device_sm_count(int* sms, int* smem_optin) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { cudaGetLastError(); return fail(ATTN_ERR_NO_DEVICE, "no CUDA device: %s", cudaGetErrorString(e)); }
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) { cudaGetLastError(); return fail(ATTN_ERR_NO_DEVICE, "no CUDA device: %s", cudaGetErrorString(e)); }
    if (major != 10) return fail(ATTN_ERR_UNSUPPORTED, "device compute capability %d.x is not 10.x", major);
    cudaDeviceGetAttribute(sms, cudaDevAttrMultiProcessorCount, dev);
    cudaDeviceGetAttribute(smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    return ATTN_OK;
}

int grid_for(long long n_work, int sm_count, const Resolved& r) {
    long long cap = sm_count;
    if (r.max_ctas > 0 && r.max_ctas < cap) cap = r.max_ctas;
    if (r.launch_mode == 1) return (int)(n_work < 2147483647LL ? n_work : 2147483647LL);  // Algorithm 3
    return (int)(n_work < cap ? n_work : cap);                                           // Algorithm 2
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int get_encoder(EncodeTiledFn* fn) {
    static EncodeTiledFn cached = nullptr;
    if (!cached) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
        if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !p) {
            cudaGetLastError();
            return fail(ATTN_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
        }
        cached = reinterpret_cast<EncodeTiledFn>(p);
    }
    *fn = cached;
    return ATTN_OK;
}

// [B*H, N, d] view, box = `cols` (64 or 32) columns x `rows` rows of one head, rows of the box swizzled over their
// own length (128 or 64 bytes), zero fill outside.
int make_map(CUtensorMap* m, const void* base, int BH, int N, int d, int rows, int dtype, int cols = 64) {
    EncodeTiledFn enc;
    int rc = get_encoder(&enc);
    if (rc) return rc;
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)BH};
    cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)N * d * 2};
    cuuint32_t box[3] = {(cuuint32_t)cols, (cuuint32_t)rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(m, dtype == ATTN_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3,
                     const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     cols == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(ATTN_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
    return ATTN_OK;
}

template <int kD, int kBlockN, int kQTiles, int kBf16>
int launch(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to, const KernelParams& kp, int grid,
           size_t smem, cudaStream_t stream) {
    auto kern = attn_fwd_kernel<kD, kBlockN, kQTiles, kBf16>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) { cudaGetLastError(); return fail(ATTN_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e)); }
    kern<<<grid, Geometry<kD, kBlockN, kQTiles>::kThreads, smem, stream>>>(tq, tk, tv, to, kp);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
    return ATTN_OK;
}

template <int kD, int kBlockN, int kQTiles>
int launch_dtype(int dtype, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to, const KernelParams& kp,
                 int grid, size_t smem, cudaStream_t stream) {
    return dtype == ATTN_BF16 ? launch<kD, kBlockN, kQTiles, 1>(tq, tk, tv, to, kp, grid, smem, stream)
                              : launch<kD, kBlockN, kQTiles, 0>(tq, tk, tv, to, kp, grid, smem, stream);
}

template <int kD>
int launch_tiles(int block_n, int q_tiles, int dtype, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                 const CUtensorMap& to, const KernelParams& kp, int grid, size_t smem, cudaStream_t stream) {
    if (block_n == 128) {
        return q_tiles == 2 ? launch_dtype<kD, 128, 2>(dtype, tq, tk, tv, to, kp, grid, smem, stream)
                            : launch_dtype<kD, 128, 1>(dtype, tq, tk, tv, to, kp, grid, smem, stream);
    }
    return q_tiles == 2 ? launch_dtype<kD, 64, 2>(dtype, tq, tk, tv, to, kp, grid, smem, stream)
                        : launch_dtype<kD, 64, 1>(dtype, tq, tk, tv, to, kp, grid, smem, stream);
}

}  // namespace

extern "C" {

const char* attn_status_string(int status) {
    switch (status) {
        case ATTN_OK: return "ok";
        case ATTN_ERR_INVALID_ARG: return "invalid argument";
        case ATTN_ERR_UNSUPPORTED: return "unsupported configuration or device";
        case ATTN_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case ATTN_ERR_NO_DEVICE: return "no CUDA device";
        case ATTN_ERR_CUDA: return "CUDA call failed";
        case ATTN_ERR_DEVICE_TIMEOUT: return "a bounded wait inside the kernel ran out";
        default: return "unknown status";
    }
}

const char* attn_last_error(void) { return g_error; }

int attn_query_plan(int B, int H, int N, int d, int causal, int dtype, const attn_fwd_opts* opts, int sm_count,
                    attn_plan* out) {
    if (!out) return fail(ATTN_ERR_INVALID_ARG, "out is null");
    int rc = check_shape(B, H, N, d, causal, dtype);
    if (rc) return rc;
    int smem_limit = kSmemOptinB200;
    if (sm_count <= 0) {
        rc = device_sm_count(&sm_count, &smem_limit);
        if (rc) return rc;
    }
    Resolved r;
    rc = resolve_opts(opts, d, smem_limit, &r);
    if (rc) return rc;
    const SchedParams sp = make_sched(B, H, N, r.q_tiles, r.block_n, causal, 0, r.head_fastest);
    out->block_m = kBlockM;
    out->block_n = r.block_n;
    out->q_tiles = r.q_tiles;
    out->rows_per_item = kBlockM * r.q_tiles;
    out->items_per_head = sp.n_q;
    out->n_work = sp.n_work;
    out->grid = grid_for(sp.n_work, sm_count, r);
    out->threads = 384;  // eight softmax warps, the producer warp, two MMA warps, one idle warp
    out->kv_stages = r.stages;
    out->smem_bytes = (int)r.smem;
    out->sm_count = sm_count;
    return ATTN_OK;
}

int attn_schedule_trace(int B, int H, int N, int d, int causal, int scan_order, int dtype, const attn_fwd_opts* opts,
                        int sm_count, attn_trace_entry* buf, size_t cap, size_t* n) {
    if (!n) return fail(ATTN_ERR_INVALID_ARG, "n is null");
    if (cap > 0 && !buf) return fail(ATTN_ERR_INVALID_ARG, "buf is null");
    if (scan_order != ATTN_SCAN_CYCLIC && scan_order != ATTN_SCAN_SAWTOOTH)
        return fail(ATTN_ERR_INVALID_ARG, "unknown scan_order %d", scan_order);
    attn_plan plan;
    int rc = attn_query_plan(B, H, N, d, causal, dtype, opts, sm_count, &plan);
    if (rc) return rc;
    const int head_fastest = opts && opts->digit_order == ATTN_HEAD_FASTEST;
    const SchedParams sp = make_sched(B, H, N, plan.q_tiles, plan.block_n, causal, scan_order == ATTN_SCAN_SAWTOOTH, head_fastest);
    size_t count = 0;
    for (int cta = 0; cta < plan.grid; ++cta) {
        int it = 0;
        for (long long k = cta; k < sp.n_work; k += plan.grid, ++it) {
            if (count < cap) {
                const WorkItem w = decode_work(sp, k, it);
                attn_trace_entry* e = &buf[count];
                e->cta = cta;
                e->iteration = it;
                e->k = k;
                e->batch = w.bh / H;
                e->head = w.bh % H;
                e->q_item = w.q_item;
                e->backward = w.backward;
                e->n_kv = w.hi;
                e->n_kv_q0 = w.hi_q[0];
                e->n_kv_q1 = w.hi_q[1];
            }
            ++count;
        }
    }
    *n = count;
    return ATTN_OK;
}

static int fwd_common(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d, float scale, int causal,
                      int scan_order, int dtype, void* stream, const attn_fwd_opts* opts, int* work_counter, size_t counter_bytes,
                      int counter_ctas_max);

int attn_fwd_ex(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d, float scale, int causal,
                int scan_order, int dtype, void* stream, const attn_fwd_opts* opts) {
    return fwd_common(q, k, v, o, B, H, N, d, scale, causal, scan_order, dtype, stream, opts, nullptr, 0, 0);
}

size_t attn_dynamic_scratch_bytes(int ctas) { return (size_t)ATTN_DYNAMIC_SCRATCH_HEADER + 4u * (size_t)(ctas > 0 ? ctas : 0); }

int attn_fwd_dynamic(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d, float scale, int causal,
                     int scan_order, int dtype, void* stream, const attn_fwd_opts* opts, void* scratch, size_t scratch_bytes) {
    if (!scratch) return fail(ATTN_ERR_INVALID_ARG, "scratch is null");
    if ((uintptr_t)scratch & 3u) return fail(ATTN_ERR_ALIGNMENT, "scratch must be 4-byte aligned");
    if (scratch_bytes < (size_t)ATTN_DYNAMIC_SCRATCH_HEADER) return fail(ATTN_ERR_INVALID_ARG, "scratch is smaller than its %d-byte header", ATTN_DYNAMIC_SCRATCH_HEADER);
    const size_t ctas_max = (scratch_bytes - ATTN_DYNAMIC_SCRATCH_HEADER) / 4;
    return fwd_common(q, k, v, o, B, H, N, d, scale, causal, scan_order, dtype, stream, opts, static_cast<int*>(scratch), scratch_bytes,
                      (int)(ctas_max < 2147483647u ? ctas_max : 2147483647u));
}

int attn_fwd_dynamic_noalloc(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d, float scale,
                             int causal, int scan_order, int dtype, void* stream, const attn_fwd_opts* opts) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { cudaGetLastError(); return fail(ATTN_ERR_NO_DEVICE, "no CUDA device: %s", cudaGetErrorString(e)); }
    if (dev < 0 || dev >= kMaxDevices) return fail(ATTN_ERR_UNSUPPORTED, "device index %d is beyond the %d this entry point keeps track of", dev, kMaxDevices);
    if (!g_noalloc_ptr[dev]) {
        // Set-up, once per device, with that device current.  In host code the array's name is only a handle for
        // this lookup, not an address a kernel could use; the lookup gives the address inside the current device.
        int* ptr = nullptr;
        e = cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch);
        if (e != cudaSuccess || !ptr) { cudaGetLastError(); return fail(ATTN_ERR_CUDA, "cudaGetSymbolAddress(scratch): %s", cudaGetErrorString(e)); }
        g_noalloc_ptr[dev] = ptr;
    }
    // fwd_common turns a launch of more than ATTN_NOALLOC_MAX_CTAS CTAs away before anything is enqueued.
    return fwd_common(q, k, v, o, B, H, N, d, scale, causal, scan_order, dtype, stream, opts, g_noalloc_ptr[dev], sizeof(g_noalloc_scratch),
                      ATTN_NOALLOC_MAX_CTAS);
}

static int fwd_common(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d, float scale, int causal,
                      int scan_order, int dtype, void* stream, const attn_fwd_opts* opts, int* work_counter, size_t counter_bytes,
                      int counter_ctas_max) {
    if (!q || !k || !v || !o) return fail(ATTN_ERR_INVALID_ARG, "q, k, v and o must be non-null");
    int rc = check_shape(B, H, N, d, causal, dtype);
    if (rc) return rc;
    if (scan_order != ATTN_SCAN_CYCLIC && scan_order != ATTN_SCAN_SAWTOOTH)
        return fail(ATTN_ERR_INVALID_ARG, "unknown scan_order %d", scan_order);
    if (!std::isfinite(scale) || !(scale > 0.f)) return fail(ATTN_ERR_INVALID_ARG, "scale must be finite and positive");
    if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)o) & 15u)
        return fail(ATTN_ERR_ALIGNMENT, "q, k, v and o must be 16-byte aligned");
    int sm_count = 0, smem_limit = 0;
    rc = device_sm_count(&sm_count, &smem_limit);
    if (rc) return rc;
    Resolved r;
    rc = resolve_opts(opts, d, smem_limit, &r);
    if (rc) return rc;

    KernelParams kp;
    // Dynamic schedule: items are claimed in index order, and under the causal mask that order runs from the last
    // (longest) Q block of a head to the first, so that the short items fill the end of the launch.
    kp.sched = make_sched(B, H, N, r.q_tiles, r.block_n, causal, scan_order == ATTN_SCAN_SAWTOOTH, r.head_fastest,
                          work_counter != nullptr && causal);
    kp.work_counter = work_counter;
    kp.scale_log2 = scale * 1.4426950408889634f;
    kp.kv_stages = r.stages;
    kp.l2_policy = r.l2_policy;
    kp.o = o;
    rc = (int)cudaGetSymbolAddress((void**)&kp.status, g_status_word);
    if (rc != 0) { cudaGetLastError(); return fail(ATTN_ERR_CUDA, "cudaGetSymbolAddress failed (%d)", rc); }
    rc = (int)cudaGetSymbolAddress((void**)&kp.cycles, g_cycles);
    if (rc != 0) { cudaGetLastError(); return fail(ATTN_ERR_CUDA, "cudaGetSymbolAddress failed (%d)", rc); }

    CUtensorMap tq, tk, tv;
    if ((rc = make_map(&tq, q, B * H, N, d, kBlockM, dtype))) return rc;
    if ((rc = make_map(&tk, k, B * H, N, d, r.block_n, dtype))) return rc;
    if ((rc = make_map(&tv, v, B * H, N, d, r.block_n, dtype))) return rc;
    // O is written through shared memory, each softmax warp storing boxes of its d/2 columns x as many rows (at most its
    // 32) as its eighth of a ring slot holds.
    CUtensorMap to;
    const int stage_row_bytes = d, stage_bytes_per_warp = r.block_n * d * 2 / 8;
    const int stage_rows = stage_bytes_per_warp / stage_row_bytes < 32 ? stage_bytes_per_warp / stage_row_bytes : 32;
    if ((rc = make_map(&to, o, B * H, N, d, stage_rows, dtype, d / 2))) return rc;

    const int grid = grid_for(kp.sched.n_work, sm_count, r);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (work_counter) {
        if (r.launch_mode != 0) return fail(ATTN_ERR_INVALID_ARG, "the dynamic schedule needs the persistent launch (launch_mode 0)");
        if (grid > counter_ctas_max)
            return fail(ATTN_ERR_INVALID_ARG, "scratch holds counters for %d CTAs, the launch has %d (need %zu bytes)", counter_ctas_max, grid,
                        (size_t)ATTN_DYNAMIC_SCRATCH_HEADER + 4u * (size_t)grid);
        (void)counter_bytes;
        cudaError_t e = cudaMemsetAsync(work_counter, 0, (size_t)ATTN_DYNAMIC_SCRATCH_HEADER + 4u * (size_t)grid, st);
        if (e != cudaSuccess) { cudaGetLastError(); return fail(ATTN_ERR_CUDA, "clearing the scratch: %s", cudaGetErrorString(e)); }
    }
    return d == 128 ? launch_tiles<128>(r.block_n, r.q_tiles, dtype, tq, tk, tv, to, kp, grid, r.smem, st)
                    : launch_tiles<64>(r.block_n, r.q_tiles, dtype, tq, tk, tv, to, kp, grid, r.smem, st);
}

int attn_fwd(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d, float scale, int causal,
             int scan_order, int dtype, void* stream) {
    return attn_fwd_ex(q, k, v, o, B, H, N, d, scale, causal, scan_order, dtype, stream, nullptr);
}

namespace {
// Streams and events of the attn_fwd_host pipeline, one set per device, created on first use.
struct HostPipe {
    bool ready = false;
    cudaStream_t up = nullptr, run = nullptr, down = nullptr;
    cudaEvent_t start = nullptr, done = nullptr, uploaded[kMaxHostChunks] = {}, computed[kMaxHostChunks] = {};
};
HostPipe g_host_pipe[kMaxDevices];
std::mutex g_host_pipe_mutex;

int host_pipe_for_current_device(HostPipe** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { cudaGetLastError(); return fail(ATTN_ERR_NO_DEVICE, "no CUDA device: %s", cudaGetErrorString(e)); }
    if (dev < 0 || dev >= kMaxDevices) return fail(ATTN_ERR_UNSUPPORTED, "device index %d is beyond the %d the host pipeline keeps track of", dev, kMaxDevices);
    std::lock_guard<std::mutex> lock(g_host_pipe_mutex);
    HostPipe& hp = g_host_pipe[dev];
    if (!hp.ready) {
        bool ok = cudaStreamCreateWithFlags(&hp.up, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&hp.run, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&hp.down, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.done, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; ok && i < kMaxHostChunks; ++i)
            ok = cudaEventCreateWithFlags(&hp.uploaded[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&hp.computed[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) { cudaGetLastError(); return fail(ATTN_ERR_CUDA, "creating the streams and events of the host pipeline failed"); }
        hp.ready = true;
    }
    *out = &hp;
    return ATTN_OK;
}
}  // namespace

int attn_fwd_host(const void* q_host, const void* k_host, const void* v_host, void* o_host, void* q_dev, void* k_dev,
                  void* v_dev, void* o_dev, int B, int H, int N, int d, float scale, int causal, int scan_order, int dtype,
                  void* stream, const attn_fwd_opts* opts) {
    if (!q_host || !k_host || !v_host || !o_host) return fail(ATTN_ERR_INVALID_ARG, "host buffers must be non-null");
    if (!q_dev || !k_dev || !v_dev || !o_dev) return fail(ATTN_ERR_INVALID_ARG, "device staging buffers must be non-null");
    int rc = check_shape(B, H, N, d, causal, dtype);
    if (rc) return rc;
    const size_t bytes = (size_t)B * H * N * d * 2;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    const long long heads = (long long)B * H;
    int chunks = opts ? opts->host_chunks : 0;
    if (chunks < 0 || chunks > kMaxHostChunks) return fail(ATTN_ERR_INVALID_ARG, "host_chunks must be in [0, %d]", kMaxHostChunks);
    if (chunks == 0) chunks = bytes > ((size_t)32 << 20) ? 8 : 1;
    if (chunks > heads) chunks = (int)heads;
    if (chunks <= 1) {
        if ((e = cudaMemcpyAsync(q_dev, q_host, bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
            (e = cudaMemcpyAsync(k_dev, k_host, bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
            (e = cudaMemcpyAsync(v_dev, v_host, bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess) {
            cudaGetLastError();
            return fail(ATTN_ERR_CUDA, "host-to-device copy: %s", cudaGetErrorString(e));
        }
        rc = attn_fwd_ex(q_dev, k_dev, v_dev, o_dev, B, H, N, d, scale, causal, scan_order, dtype, stream, opts);
        if (rc) return rc;
        if ((e = cudaMemcpyAsync(o_host, o_dev, bytes, cudaMemcpyDeviceToHost, st)) != cudaSuccess) {
            cudaGetLastError();
            return fail(ATTN_ERR_CUDA, "device-to-host copy: %s", cudaGetErrorString(e));
        }
        return ATTN_OK;
    }
    // Pipeline over groups of heads: upload, kernel and download of successive groups overlap on three streams.
    HostPipe* hp = nullptr;
    if ((rc = host_pipe_for_current_device(&hp))) return rc;
    const size_t head_bytes = (size_t)N * d * 2;
    auto fail_cuda = [&](const char* what) { cudaGetLastError(); return fail(ATTN_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e)); };
    if ((e = cudaEventRecord(hp->start, st)) != cudaSuccess) return fail_cuda("cudaEventRecord");
    if ((e = cudaStreamWaitEvent(hp->up, hp->start, 0)) != cudaSuccess || (e = cudaStreamWaitEvent(hp->run, hp->start, 0)) != cudaSuccess ||
        (e = cudaStreamWaitEvent(hp->down, hp->start, 0)) != cudaSuccess)
        return fail_cuda("cudaStreamWaitEvent");
    long long h0 = 0;
    for (int c = 0; c < chunks; ++c) {
        const long long n_heads = heads / chunks + (c < heads % chunks ? 1 : 0);
        const size_t off = (size_t)h0 * head_bytes, len = (size_t)n_heads * head_bytes;
        const uint8_t *qh = (const uint8_t*)q_host + off, *kh = (const uint8_t*)k_host + off, *vh = (const uint8_t*)v_host + off;
        uint8_t *qd = (uint8_t*)q_dev + off, *kd = (uint8_t*)k_dev + off, *vd = (uint8_t*)v_dev + off, *od = (uint8_t*)o_dev + off;
        if ((e = cudaMemcpyAsync(qd, qh, len, cudaMemcpyHostToDevice, hp->up)) != cudaSuccess ||
            (e = cudaMemcpyAsync(kd, kh, len, cudaMemcpyHostToDevice, hp->up)) != cudaSuccess ||
            (e = cudaMemcpyAsync(vd, vh, len, cudaMemcpyHostToDevice, hp->up)) != cudaSuccess)
            return fail_cuda("host-to-device copy");
        if ((e = cudaEventRecord(hp->uploaded[c], hp->up)) != cudaSuccess || (e = cudaStreamWaitEvent(hp->run, hp->uploaded[c], 0)) != cudaSuccess)
            return fail_cuda("cudaEventRecord");
        rc = attn_fwd_ex(qd, kd, vd, od, 1, (int)n_heads, N, d, scale, causal, scan_order, dtype, hp->run, opts);
        if (rc) return rc;
        if ((e = cudaEventRecord(hp->computed[c], hp->run)) != cudaSuccess || (e = cudaStreamWaitEvent(hp->down, hp->computed[c], 0)) != cudaSuccess)
            return fail_cuda("cudaEventRecord");
        if ((e = cudaMemcpyAsync((uint8_t*)o_host + off, od, len, cudaMemcpyDeviceToHost, hp->down)) != cudaSuccess)
            return fail_cuda("device-to-host copy");
        h0 += n_heads;
    }
    if ((e = cudaEventRecord(hp->done, hp->down)) != cudaSuccess || (e = cudaStreamWaitEvent(st, hp->done, 0)) != cudaSuccess)
        return fail_cuda("cudaEventRecord");
    return ATTN_OK;
}

int attn_last_kernel_cycles(unsigned long long* cycles) {
    if (!cycles) return fail(ATTN_ERR_INVALID_ARG, "cycles is null");
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { cudaGetLastError(); return fail(ATTN_ERR_CUDA, "cudaDeviceSynchronize: %s", cudaGetErrorString(e)); }
    e = cudaMemcpyFromSymbol(cycles, g_cycles, sizeof(unsigned long long));
    if (e != cudaSuccess) { cudaGetLastError(); return fail(ATTN_ERR_CUDA, "reading the cycle count: %s", cudaGetErrorString(e)); }
    return ATTN_OK;
}

#ifdef SAW_PROFILE
/* Profiling builds only: copies the per-CTA phase table (256 x 32 cycle counts) to `out` after a device sync. */
int attn_debug_profile(unsigned long long* out) {
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpyFromSymbol(out, sawtooth::g_profile, sizeof(unsigned long long) * 256 * 32);
    if (e != cudaSuccess) { cudaGetLastError(); return fail(ATTN_ERR_CUDA, "reading the profile table: %s", cudaGetErrorString(e)); }
    return ATTN_OK;
}
#endif

int attn_device_status(int* code) {
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { cudaGetLastError(); return fail(ATTN_ERR_CUDA, "cudaDeviceSynchronize: %s", cudaGetErrorString(e)); }
    int word = 0;
    e = cudaMemcpyFromSymbol(&word, g_status_word, sizeof(int));
    if (e != cudaSuccess) { cudaGetLastError(); return fail(ATTN_ERR_CUDA, "reading the status word: %s", cudaGetErrorString(e)); }
    if (code) *code = word;
    if (word != 0) {
        const int zero = 0;
        cudaMemcpyToSymbol(g_status_word, &zero, sizeof(int));
        return fail(ATTN_ERR_DEVICE_TIMEOUT, "kernel wait site %d ran out of time", word);
    }
    return ATTN_OK;
}

}  // extern "C"
