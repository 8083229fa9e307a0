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
constexpr int kMaxHostChunks = 32;
constexpr int kSmemOptinB200 = 232448;  // 227 KiB of dynamic shared memory per CTA on sm_100
constexpr int kKernelVariants = 16;     // d x block_n x q_tiles x dtype

// What the library knows about a device, looked up once (under the mutex) on the first call that has it current:
// its size, the device addresses of the library's own __device__ variables there, and which kernel variants have had
// their dynamic shared memory limit raised.  Readers take a copy under the same mutex.
struct DeviceState {
    bool ready = false;
    int sm_count = 0, smem_optin = 0;
    int* status = nullptr;
    unsigned long long* cycles = nullptr;
    int* noalloc_scratch = nullptr;
    unsigned smem_raised = 0;   // bit v: variant v of the kernel may use smem_optin bytes
};
DeviceState g_device[kMaxDevices];
std::mutex g_device_mutex;

struct Resolved {
    int block_n, q_tiles, stages, head_fastest, launch_mode, l2_policy, max_ctas, pairing, check_mode, kv_heads, layout;
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

// `dynamic`: the call uses the dynamic schedule (items are claimed one by one, so there are no pairs).
int resolve_opts(const attn_fwd_opts* o, int d, int H, int causal, bool dynamic, int smem_limit, Resolved* r) {
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
    if (z.pairing < ATTN_PAIR_DEFAULT || z.pairing > ATTN_PAIR_ADJACENT) return fail(ATTN_ERR_INVALID_ARG, "unknown pairing %d", z.pairing);
    if (z.check_mode != 0 && z.check_mode != 1) return fail(ATTN_ERR_INVALID_ARG, "check_mode must be 0 or 1");
    if (dynamic && z.pairing > ATTN_PAIR_NONE) return fail(ATTN_ERR_INVALID_ARG, "the dynamic schedule claims single work items: pairing must be left at its default or be ATTN_PAIR_NONE");
    // Default: mirrored pairs under the causal mask (every unit of the static walk then takes the same time), none otherwise.
    r->pairing = dynamic ? kPairNone
               : z.pairing == ATTN_PAIR_DEFAULT ? (causal ? kPairMirrored : kPairNone)
               : z.pairing == ATTN_PAIR_NONE ? kPairNone : z.pairing == ATTN_PAIR_MIRRORED ? kPairMirrored : kPairAdjacent;
    r->check_mode = z.check_mode;
    if (z.kv_heads < 0 || (z.kv_heads > 0 && (z.kv_heads > H || H % z.kv_heads != 0)))
        return fail(ATTN_ERR_INVALID_ARG, "kv_heads (%d) must divide the number of query heads (%d)", z.kv_heads, H);
    r->kv_heads = z.kv_heads ? z.kv_heads : H;
    if (z.layout != ATTN_LAYOUT_BHND && z.layout != ATTN_LAYOUT_BNHD) return fail(ATTN_ERR_INVALID_ARG, "unknown layout %d", z.layout);
    r->layout = z.layout;
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

// The current device's entry of g_device, filled on first use.  *dev_out gets the device index.
int current_device(DeviceState* out, int* dev_out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { cudaGetLastError(); return fail(ATTN_ERR_NO_DEVICE, "no CUDA device: %s", cudaGetErrorString(e)); }
    if (dev < 0 || dev >= kMaxDevices) return fail(ATTN_ERR_UNSUPPORTED, "device index %d is beyond the %d the library keeps track of", dev, kMaxDevices);
    std::lock_guard<std::mutex> lock(g_device_mutex);
    DeviceState& ds = g_device[dev];
    if (!ds.ready) {
        int major = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) { cudaGetLastError(); return fail(ATTN_ERR_NO_DEVICE, "no CUDA device: %s", cudaGetErrorString(e)); }
        if (major != 10) return fail(ATTN_ERR_UNSUPPORTED, "device compute capability %d.x is not 10.x", major);
        cudaDeviceGetAttribute(&ds.sm_count, cudaDevAttrMultiProcessorCount, dev);
        cudaDeviceGetAttribute(&ds.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
        // In host code the names of __device__ variables are only handles for this lookup, not addresses a kernel could
        // use; the lookup gives the address inside the current device.
        if ((e = cudaGetSymbolAddress((void**)&ds.status, g_status_word)) != cudaSuccess ||
            (e = cudaGetSymbolAddress((void**)&ds.cycles, g_cycles)) != cudaSuccess ||
            (e = cudaGetSymbolAddress((void**)&ds.noalloc_scratch, g_noalloc_scratch)) != cudaSuccess ||
            !ds.status || !ds.cycles || !ds.noalloc_scratch) {
            cudaGetLastError();
            return fail(ATTN_ERR_CUDA, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        }
        ds.ready = true;
    }
    *out = ds;
    if (dev_out) *dev_out = dev;
    return ATTN_OK;
}

// n_units: work items, or pairs of them (what one trip of a CTA's loop handles).
int grid_for(long long n_units, int sm_count, const Resolved& r) {
    long long cap = sm_count;
    if (r.max_ctas > 0 && r.max_ctas < cap) cap = r.max_ctas;
    if (r.launch_mode == 1) return (int)(n_units < 2147483647LL ? n_units : 2147483647LL);  // Algorithm 3
    return (int)(n_units < cap ? n_units : cap);                                            // Algorithm 2
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

// [B, heads, N, d] view of a tensor stored as [B, heads, N, d] (layout 0) or [B, N, heads, d] (layout 1); dimensions from
// the innermost: d, N, heads, B.  Box = 64 columns x `rows` rows of one head, 128-byte swizzle, zero fill outside.
int make_map(CUtensorMap* m, const void* base, int B, int heads, int N, int d, int rows, int dtype, int layout) {
    EncodeTiledFn enc;
    int rc = get_encoder(&enc);
    if (rc) return rc;
    cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)heads, (cuuint64_t)B};
    const cuuint64_t row = (cuuint64_t)d * 2;
    cuuint64_t strides[3];
    if (layout == 0) { strides[0] = row; strides[1] = row * N; strides[2] = row * N * heads; }
    else { strides[0] = row * heads; strides[1] = row; strides[2] = row * heads * N; }
    cuuint32_t box[4] = {64, (cuuint32_t)rows, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(m, dtype == ATTN_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4,
                     const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(ATTN_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
    return ATTN_OK;
}

// The four tensor maps of a call are a pure function of (pointers, shape, type, tile shape); the last few a host
// thread built are kept, so that a caller who launches on the same buffers again and again pays for the encoding once.
struct MapKey {
    const void *q, *k, *v, *o;
    int B, H, H_kv, N, d, dtype, block_n, stage_rows, layout;
    bool operator==(const MapKey& x) const {
        return q == x.q && k == x.k && v == x.v && o == x.o && B == x.B && H == x.H && H_kv == x.H_kv && N == x.N && d == x.d &&
               dtype == x.dtype && block_n == x.block_n && stage_rows == x.stage_rows && layout == x.layout;
    }
};
struct MapSet { MapKey key; CUtensorMap tq, tk, tv, to; bool valid = false; };
constexpr int kMapCacheSize = 8;
thread_local MapSet g_maps[kMapCacheSize];
thread_local int g_maps_next = 0;

int maps_for(const MapKey& key, const MapSet** out) {
    for (int i = 0; i < kMapCacheSize; ++i)
        if (g_maps[i].valid && g_maps[i].key == key) { *out = &g_maps[i]; return ATTN_OK; }
    MapSet& m = g_maps[g_maps_next];
    m.valid = false;
    int rc;
    if ((rc = make_map(&m.tq, key.q, key.B, key.H, key.N, key.d, kBlockM, key.dtype, key.layout))) return rc;
    if ((rc = make_map(&m.tk, key.k, key.B, key.H_kv, key.N, key.d, key.block_n, key.dtype, key.layout))) return rc;
    if ((rc = make_map(&m.tv, key.v, key.B, key.H_kv, key.N, key.d, key.block_n, key.dtype, key.layout))) return rc;
    // O is written through shared memory in boxes of 64 columns x as many rows as one warp's share of a ring slot holds.
    if ((rc = make_map(&m.to, key.o, key.B, key.H, key.N, key.d, key.stage_rows, key.dtype, key.layout))) return rc;
    m.key = key;
    m.valid = true;
    g_maps_next = (g_maps_next + 1) % kMapCacheSize;
    *out = &m;
    return ATTN_OK;
}

template <int kD, int kBlockN, int kQTiles, int kBf16>
int launch(int dev, const DeviceState& ds, const MapSet& m, const KernelParams& kp, int grid, size_t smem, cudaStream_t stream) {
    auto kern = attn_fwd_kernel<kD, kBlockN, kQTiles, kBf16>;
    constexpr int variant = ((kD == 128) << 3) | ((kBlockN == 128) << 2) | ((kQTiles == 2) << 1) | kBf16;
    static_assert(variant < kKernelVariants, "variant index");
    if (!(ds.smem_raised & (1u << variant))) {
        // Once per device and kernel variant: allow the kernel the device's whole opt-in shared memory.
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ds.smem_optin);
        if (e != cudaSuccess) { cudaGetLastError(); return fail(ATTN_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e)); }
        std::lock_guard<std::mutex> lock(g_device_mutex);
        g_device[dev].smem_raised |= 1u << variant;
    }
    kern<<<grid, Geometry<kD, kBlockN, kQTiles>::kThreads, smem, stream>>>(m.tq, m.tk, m.tv, m.to, kp);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
    return ATTN_OK;
}

template <int kD, int kBlockN, int kQTiles>
int launch_dtype(int dtype, int dev, const DeviceState& ds, const MapSet& m, const KernelParams& kp, int grid, size_t smem, cudaStream_t stream) {
    return dtype == ATTN_BF16 ? launch<kD, kBlockN, kQTiles, 1>(dev, ds, m, kp, grid, smem, stream)
                              : launch<kD, kBlockN, kQTiles, 0>(dev, ds, m, kp, grid, smem, stream);
}

template <int kD>
int launch_tiles(int block_n, int q_tiles, int dtype, int dev, const DeviceState& ds, const MapSet& m, const KernelParams& kp, int grid,
                 size_t smem, cudaStream_t stream) {
    if (block_n == 128) {
        return q_tiles == 2 ? launch_dtype<kD, 128, 2>(dtype, dev, ds, m, kp, grid, smem, stream)
                            : launch_dtype<kD, 128, 1>(dtype, dev, ds, m, kp, grid, smem, stream);
    }
    return q_tiles == 2 ? launch_dtype<kD, 64, 2>(dtype, dev, ds, m, kp, grid, smem, stream)
                        : launch_dtype<kD, 64, 1>(dtype, dev, ds, m, kp, grid, smem, stream);
}

// Reads and clears the current device's status word after a device synchronisation.
int read_status(int* code) {
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
        DeviceState ds;
        rc = current_device(&ds, nullptr);
        if (rc) return rc;
        sm_count = ds.sm_count;
        smem_limit = ds.smem_optin;
    }
    Resolved r;
    rc = resolve_opts(opts, d, H, causal, false, smem_limit, &r);
    if (rc) return rc;
    const SchedParams sp = make_sched(B, H, N, r.q_tiles, r.block_n, causal, 0, r.head_fastest, 0, r.pairing);
    out->block_m = kBlockM;
    out->block_n = r.block_n;
    out->q_tiles = r.q_tiles;
    out->rows_per_item = kBlockM * r.q_tiles;
    out->items_per_head = sp.n_q;
    out->n_work = sp.n_work;
    out->grid = grid_for(sp.n_units, sm_count, r);
    out->threads = r.q_tiles * 128 + 128;
    out->kv_stages = r.stages;
    out->smem_bytes = (int)r.smem;
    out->sm_count = sm_count;
    out->pairing = r.pairing == kPairNone ? ATTN_PAIR_NONE : r.pairing == kPairMirrored ? ATTN_PAIR_MIRRORED : ATTN_PAIR_ADJACENT;
    out->n_units = sp.n_units;
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
    const int pairing = plan.pairing == ATTN_PAIR_NONE ? kPairNone : plan.pairing == ATTN_PAIR_MIRRORED ? kPairMirrored : kPairAdjacent;
    const SchedParams sp = make_sched(B, H, N, plan.q_tiles, plan.block_n, causal, scan_order == ATTN_SCAN_SAWTOOTH, head_fastest, 0, pairing);
    const int members = pairing == kPairNone ? 1 : 2;
    size_t count = 0;
    for (int cta = 0; cta < plan.grid; ++cta) {
        int it = 0;
        for (int slot = 0;; ++slot) {
            const Slot sl = static_slot(sp, cta, plan.grid, slot);
            if (sl.kind == kSlotEnd) break;
            if (sl.kind == kSlotEmpty) continue;
            if (count < cap) {
                const WorkItem w = make_item(sp, sl.bh, sl.q_item, it);
                attn_trace_entry* e = &buf[count];
                e->cta = cta;
                e->iteration = it;
                e->k = (long long)cta + (long long)(slot / members) * plan.grid;
                e->batch = w.bh / H;
                e->head = w.bh % H;
                e->q_item = w.q_item;
                e->backward = w.backward;
                e->n_kv = w.hi;
                e->n_kv_q0 = w.hi_q[0];
                e->n_kv_q1 = w.hi_q[1];
                e->member = slot % members;
            }
            ++count;
            ++it;
        }
    }
    *n = count;
    return ATTN_OK;
}

int attn_dynamic_claim_trace(int B, int H, int N, int d, int causal, int scan_order, int dtype, const attn_fwd_opts* opts,
                             int sm_count, attn_trace_entry* buf, size_t cap, size_t* n) {
    if (!n) return fail(ATTN_ERR_INVALID_ARG, "n is null");
    if (cap > 0 && !buf) return fail(ATTN_ERR_INVALID_ARG, "buf is null");
    if (scan_order != ATTN_SCAN_CYCLIC && scan_order != ATTN_SCAN_SAWTOOTH)
        return fail(ATTN_ERR_INVALID_ARG, "unknown scan_order %d", scan_order);
    attn_fwd_opts single;
    memset(&single, 0, sizeof(single));
    if (opts) single = *opts;
    single.pairing = ATTN_PAIR_NONE;   // single items are claimed
    attn_plan plan;
    int rc = attn_query_plan(B, H, N, d, causal, dtype, &single, sm_count, &plan);
    if (rc) return rc;
    const SchedParams sp = make_sched(B, H, N, plan.q_tiles, plan.block_n, causal, scan_order == ATTN_SCAN_SAWTOOTH,
                                      single.digit_order == ATTN_HEAD_FASTEST, causal ? 1 : 0, kPairNone);
    size_t count = 0;
    for (long long claim = 0;; ++claim) {
        const Slot sl = claimed_slot(sp, claim);
        if (sl.kind == kSlotEnd) break;
        if (count < cap) {
            const int round = (int)(claim / plan.grid);
            const WorkItem w = make_item(sp, sl.bh, sl.q_item, round);
            attn_trace_entry* e = &buf[count];
            e->cta = -1;
            e->iteration = round;
            e->k = claim;
            e->batch = w.bh / H;
            e->head = w.bh % H;
            e->q_item = w.q_item;
            e->backward = w.backward;
            e->n_kv = w.hi;
            e->n_kv_q0 = w.hi_q[0];
            e->n_kv_q1 = w.hi_q[1];
            e->member = 0;
        }
        ++count;
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
    // The first call on a device looks the scratch array's address up there (see current_device); later calls reuse it.
    DeviceState ds;
    int rc = current_device(&ds, nullptr);
    if (rc) return rc;
    // fwd_common turns a launch of more than ATTN_NOALLOC_MAX_CTAS CTAs away before anything is enqueued.
    return fwd_common(q, k, v, o, B, H, N, d, scale, causal, scan_order, dtype, stream, opts, ds.noalloc_scratch, sizeof(g_noalloc_scratch),
                      ATTN_NOALLOC_MAX_CTAS);
}

// Everything that can be refused is refused here, before anything is enqueued.
struct Checked {
    Resolved r;
    DeviceState ds;
    int dev;
};
static int check_call(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d, float scale, int causal,
                      int scan_order, int dtype, const attn_fwd_opts* opts, bool dynamic, Checked* c) {
    if (!q || !k || !v || !o) return fail(ATTN_ERR_INVALID_ARG, "q, k, v and o must be non-null");
    int rc = check_shape(B, H, N, d, causal, dtype);
    if (rc) return rc;
    if (scan_order != ATTN_SCAN_CYCLIC && scan_order != ATTN_SCAN_SAWTOOTH)
        return fail(ATTN_ERR_INVALID_ARG, "unknown scan_order %d", scan_order);
    if (!std::isfinite(scale)) return fail(ATTN_ERR_INVALID_ARG, "scale must be finite");
    if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)o) & 15u)
        return fail(ATTN_ERR_ALIGNMENT, "q, k, v and o must be 16-byte aligned");
    if (opts && opts->lse && ((uintptr_t)opts->lse & 3u)) return fail(ATTN_ERR_ALIGNMENT, "opts->lse must be 4-byte aligned");
    rc = current_device(&c->ds, &c->dev);
    if (rc) return rc;
    return resolve_opts(opts, d, H, causal, dynamic, c->ds.smem_optin, &c->r);
}

static int fwd_common(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d, float scale, int causal,
                      int scan_order, int dtype, void* stream, const attn_fwd_opts* opts, int* work_counter, size_t counter_bytes,
                      int counter_ctas_max) {
    Checked c;
    int rc = check_call(q, k, v, o, B, H, N, d, scale, causal, scan_order, dtype, opts, work_counter != nullptr, &c);
    if (rc) return rc;
    const Resolved& r = c.r;

    KernelParams kp;
    // Dynamic schedule: items are claimed in index order, and under the causal mask that order runs from the last
    // (longest) Q block of a head to the first, so that the short items fill the end of the launch.
    kp.sched = make_sched(B, H, N, r.q_tiles, r.block_n, causal, scan_order == ATTN_SCAN_SAWTOOTH, r.head_fastest,
                          work_counter != nullptr && causal, r.pairing);
    kp.work_counter = work_counter;
    // softmax(scale * s) is computed as 2^(|scale| log2(e) * (+-s) - m).  A scale of exactly zero (every visible key gets
    // the same weight) runs as the smallest positive scale: the products then vanish against m, masked keys keep -inf.
    const float mag = scale == 0.f ? 1e-30f : std::fabs(scale);
    kp.scale_log2 = mag * 1.4426950408889634f;
    kp.negate = scale < 0.f;
    kp.kv_stages = r.stages;
    kp.kv_heads = r.kv_heads;
    kp.l2_policy = r.l2_policy;
    kp.o = o;
    kp.lse = opts ? opts->lse : nullptr;
    kp.status = c.ds.status;
    kp.cycles = c.ds.cycles;

    MapKey key;
    key.q = q; key.k = k; key.v = v; key.o = o;
    key.B = B; key.H = H; key.H_kv = r.kv_heads; key.layout = r.layout; key.N = N; key.d = d; key.dtype = dtype; key.block_n = r.block_n;
    key.stage_rows = (r.block_n * d * 2 / 2 / 4) / 128 < 32 ? (r.block_n * d * 2 / 2 / 4) / 128 : 32;
    const MapSet* maps = nullptr;
    if ((rc = maps_for(key, &maps))) return rc;

    const int grid = grid_for(kp.sched.n_units, c.ds.sm_count, r);
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
    rc = d == 128 ? launch_tiles<128>(r.block_n, r.q_tiles, dtype, c.dev, c.ds, *maps, kp, grid, r.smem, st)
                  : launch_tiles<64>(r.block_n, r.q_tiles, dtype, c.dev, c.ds, *maps, kp, grid, r.smem, st);
    if (rc) return rc;
    // check_mode: wait for the device and report a wait that ran out inside the kernel as this call's status.
    return r.check_mode ? read_status(nullptr) : ATTN_OK;
}

int attn_fwd(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int d, float scale, int causal,
             int scan_order, int dtype, void* stream) {
    return attn_fwd_ex(q, k, v, o, B, H, N, d, scale, causal, scan_order, dtype, stream, nullptr);
}

namespace {
// Streams and events of the attn_fwd_host pipeline, one set per device, created on first use.  One call at a time
// enqueues on a device's set: the set's mutex is held from the first event record to the last.
struct HostPipe {
    std::mutex busy;
    bool ready = false;
    cudaStream_t up = nullptr, run[2] = {nullptr, nullptr}, down = nullptr;
    cudaEvent_t start = nullptr, done_up = nullptr, done_run[2] = {nullptr, nullptr}, done_down = nullptr;
    cudaEvent_t uploaded[kMaxHostChunks] = {}, computed[kMaxHostChunks] = {};
};
HostPipe g_host_pipe[kMaxDevices];

// Called with hp.busy held.
int prepare_host_pipe(HostPipe& hp) {
    if (hp.ready) return ATTN_OK;
    bool ok = cudaStreamCreateWithFlags(&hp.up, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&hp.run[0], cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&hp.run[1], cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&hp.down, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.done_up, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.done_run[0], cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.done_run[1], cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.done_down, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < kMaxHostChunks; ++i)
        ok = cudaEventCreateWithFlags(&hp.uploaded[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&hp.computed[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return fail(ATTN_ERR_CUDA, "creating the streams and events of the host pipeline failed"); }
    hp.ready = true;
    return ATTN_OK;
}

// Groups of heads for attn_fwd_host: host_chunks equal ones (the first ones a head larger when it does not divide), or,
// left to the library, one group per 16 MiB of a tensor once the tensor exceeds 32 MiB (kMaxHostChunks at most, a head
// at least).  Small equal groups: upload and kernel take about as long as each other on a PCIe 5 link, so what counts
// is that the first kernel starts early and that no kernel waits for a long upload.
int host_groups(long long heads, size_t head_bytes, int host_chunks, long long* group) {
    long long chunks = host_chunks;
    if (chunks == 0) {
        const size_t bytes = (size_t)heads * head_bytes;
        chunks = bytes > ((size_t)32 << 20) ? (long long)(bytes >> 24) : 1;
        if (chunks > kMaxHostChunks) chunks = kMaxHostChunks;
    }
    if (chunks > heads) chunks = heads;
    for (long long ch = 0; ch < chunks; ++ch) group[ch] = heads / chunks + (ch < heads % chunks ? 1 : 0);
    return (int)chunks;
}
}  // namespace

int attn_host_groups(long long heads, size_t head_bytes, int host_chunks, long long* sizes, int* n) {
    if (heads <= 0 || head_bytes == 0 || !sizes || !n) return fail(ATTN_ERR_INVALID_ARG, "heads and head_bytes must be positive, sizes and n non-null");
    if (host_chunks < 0 || host_chunks > kMaxHostChunks) return fail(ATTN_ERR_INVALID_ARG, "host_chunks must be in [0, %d]", kMaxHostChunks);
    *n = host_groups(heads, head_bytes, host_chunks, sizes);
    return ATTN_OK;
}

int attn_fwd_host(const void* q_host, const void* k_host, const void* v_host, void* o_host, void* q_dev, void* k_dev,
                  void* v_dev, void* o_dev, int B, int H, int N, int d, float scale, int causal, int scan_order, int dtype,
                  void* stream, const attn_fwd_opts* opts) {
    if (!q_host || !k_host || !v_host || !o_host) return fail(ATTN_ERR_INVALID_ARG, "host buffers must be non-null");
    // Every argument and option is checked before the first copy is enqueued.
    Checked c;
    int rc = check_call(q_dev, k_dev, v_dev, o_dev, B, H, N, d, scale, causal, scan_order, dtype, opts, false, &c);
    if (rc) return rc;
    if (c.r.check_mode) return fail(ATTN_ERR_INVALID_ARG, "check_mode would make attn_fwd_host wait inside its pipeline: call attn_device_status afterwards instead");
    if (c.r.layout != ATTN_LAYOUT_BHND) return fail(ATTN_ERR_UNSUPPORTED, "attn_fwd_host cuts the heads into contiguous groups: layout must be ATTN_LAYOUT_BHND");
    if (c.r.kv_heads != H) return fail(ATTN_ERR_UNSUPPORTED, "attn_fwd_host cuts the heads into groups and takes as many K/V heads as query heads (kv_heads = 0)");
    attn_fwd_opts inner;
    memset(&inner, 0, sizeof(inner));
    if (opts) inner = *opts;
    inner.lse = nullptr;   // the groups of heads below are separate launches with their own [heads, N] numbering
    const size_t bytes = (size_t)B * H * N * d * 2;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaSuccess;
    const long long heads = (long long)B * H;
    long long group[kMaxHostChunks];
    const int chunks = host_groups(heads, (size_t)N * d * 2, inner.host_chunks, group);
    if (chunks <= 1) {
        if ((e = cudaMemcpyAsync(q_dev, q_host, bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
            (e = cudaMemcpyAsync(k_dev, k_host, bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
            (e = cudaMemcpyAsync(v_dev, v_host, bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess) {
            cudaGetLastError();
            return fail(ATTN_ERR_CUDA, "host-to-device copy: %s", cudaGetErrorString(e));
        }
        rc = attn_fwd_ex(q_dev, k_dev, v_dev, o_dev, B, H, N, d, scale, causal, scan_order, dtype, stream, &inner);
        if (rc) return rc;
        if ((e = cudaMemcpyAsync(o_host, o_dev, bytes, cudaMemcpyDeviceToHost, st)) != cudaSuccess) {
            cudaGetLastError();
            return fail(ATTN_ERR_CUDA, "device-to-host copy: %s", cudaGetErrorString(e));
        }
        return ATTN_OK;
    }
    // Pipeline over groups of heads: upload, kernel and download of successive groups overlap.  The kernels alternate
    // between two streams: a group's launch rarely fills its last round of work items, and the next group's CTAs move
    // onto the SMs that fall idle (the two kernels share nothing but read-only options).
    HostPipe& hp = g_host_pipe[c.dev];
    std::lock_guard<std::mutex> lock(hp.busy);
    if ((rc = prepare_host_pipe(hp))) return rc;
    const size_t head_bytes = (size_t)N * d * 2;
    const char* what = "";
    if ((e = cudaEventRecord(hp.start, st)) != cudaSuccess) { cudaGetLastError(); return fail(ATTN_ERR_CUDA, "cudaEventRecord: %s", cudaGetErrorString(e)); }
    // From here on the side streams may hold work: whatever happens, `stream` is made to wait for all three before returning.
    bool failed = false;
    auto check = [&](cudaError_t err, const char* where) {
        if (err != cudaSuccess && !failed) { failed = true; e = err; what = where; cudaGetLastError(); }
        return err == cudaSuccess;
    };
    check(cudaStreamWaitEvent(hp.up, hp.start, 0), "cudaStreamWaitEvent");
    check(cudaStreamWaitEvent(hp.run[0], hp.start, 0), "cudaStreamWaitEvent");
    check(cudaStreamWaitEvent(hp.run[1], hp.start, 0), "cudaStreamWaitEvent");
    check(cudaStreamWaitEvent(hp.down, hp.start, 0), "cudaStreamWaitEvent");
    long long h0 = 0;
    for (int ch = 0; ch < chunks && !failed && rc == 0; ++ch) {
        const long long n_heads = group[ch];
        cudaStream_t run = hp.run[ch & 1];
        const size_t off = (size_t)h0 * head_bytes, len = (size_t)n_heads * head_bytes;
        const uint8_t *qh = (const uint8_t*)q_host + off, *kh = (const uint8_t*)k_host + off, *vh = (const uint8_t*)v_host + off;
        uint8_t *qd = (uint8_t*)q_dev + off, *kd = (uint8_t*)k_dev + off, *vd = (uint8_t*)v_dev + off, *od = (uint8_t*)o_dev + off;
        if (!check(cudaMemcpyAsync(qd, qh, len, cudaMemcpyHostToDevice, hp.up), "host-to-device copy") ||
            !check(cudaMemcpyAsync(kd, kh, len, cudaMemcpyHostToDevice, hp.up), "host-to-device copy") ||
            !check(cudaMemcpyAsync(vd, vh, len, cudaMemcpyHostToDevice, hp.up), "host-to-device copy") ||
            !check(cudaEventRecord(hp.uploaded[ch], hp.up), "cudaEventRecord") ||
            !check(cudaStreamWaitEvent(run, hp.uploaded[ch], 0), "cudaStreamWaitEvent"))
            break;
        rc = attn_fwd_ex(qd, kd, vd, od, 1, (int)n_heads, N, d, scale, causal, scan_order, dtype, run, &inner);
        if (rc) break;
        if (!check(cudaEventRecord(hp.computed[ch], run), "cudaEventRecord") ||
            !check(cudaStreamWaitEvent(hp.down, hp.computed[ch], 0), "cudaStreamWaitEvent") ||
            !check(cudaMemcpyAsync((uint8_t*)o_host + off, od, len, cudaMemcpyDeviceToHost, hp.down), "device-to-host copy"))
            break;
        h0 += n_heads;
    }
    // Join: `stream` continues only after everything enqueued on the three side streams, on success and on failure alike.
    check(cudaEventRecord(hp.done_up, hp.up), "cudaEventRecord");
    check(cudaEventRecord(hp.done_run[0], hp.run[0]), "cudaEventRecord");
    check(cudaEventRecord(hp.done_run[1], hp.run[1]), "cudaEventRecord");
    check(cudaEventRecord(hp.done_down, hp.down), "cudaEventRecord");
    check(cudaStreamWaitEvent(st, hp.done_up, 0), "cudaStreamWaitEvent");
    check(cudaStreamWaitEvent(st, hp.done_run[0], 0), "cudaStreamWaitEvent");
    check(cudaStreamWaitEvent(st, hp.done_run[1], 0), "cudaStreamWaitEvent");
    check(cudaStreamWaitEvent(st, hp.done_down, 0), "cudaStreamWaitEvent");
    if (rc) return rc;   // attn_fwd_ex's own message stands
    if (failed) return fail(ATTN_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
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

int attn_device_status(int* code) { return read_status(code); }

}  // extern "C"
