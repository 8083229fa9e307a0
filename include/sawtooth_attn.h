/*
 * sawtooth_attn -- FlashAttention forward pass for NVIDIA B200 (sm_100a) with the paper's
 * Sawtooth Wavefront Reordering of the K/V scan.  C ABI; no C++ types or exceptions cross it.
 *
 * What is computed (Eq. 1 of the paper; `scale` is the factor Algorithm 1 multiplies S by, 1/sqrt(d)
 * in Eq. 1): for every batch b, head h and query row i,
 *
 *     O[b,h,i,:] = sum_j softmax_j( scale * Q[b,h,i,:] . K[b,h,j,:] ) * V[b,h,j,:]
 *
 * over the keys j the row may see: all N of them, or, under the causal mask, j <= i.
 *
 * How (Algorithms 1, 2 and 4): a persistent grid of G = min(#work items, #SMs) CTAs walks the work
 * items k = blockIdx.x, += G; an item is a block of W query rows of one (b, h) that stays resident in
 * shared memory while the K/V tiles of that head are streamed past it, with an online softmax.  In
 * the cyclic order every item scans its K/V tiles first to last; in the sawtooth order a CTA scans
 * first to last on its even iterations and last to first on its odd ones, so that the tiles it
 * touched last are the ones it, and the CTAs running beside it, touch next, while they are still
 * in L2.  Both orders give the same result up to the rounding order of the running sums.
 *
 * Layout: q, k, v, o are contiguous row-major [B, H, N, d] arrays (d fastest) of 16-bit elements,
 * all of the same type (IEEE fp16 or bfloat16); N_q = N_k = N.  (With opts->kv_heads set, k and v are
 * [B, kv_heads, N, d] and groups of H / kv_heads query heads share a K/V head; with opts->layout =
 * ATTN_LAYOUT_BNHD all four are [B, N, heads, d].)  Products accumulate in fp32; the
 * probabilities are rounded to the 16-bit type before the second product; O is rounded once at the
 * end.  Supported: d in {64, 128}; any B, H, N >= 1 with B*H <= 2^31-1 and N <= 2^24; scale finite
 * (any sign; zero gives every visible key the same weight).  Every base pointer must be 16-byte aligned.  `o` must
 * not overlap q, k or v.
 *
 * Ownership: the caller owns every buffer; the library allocates no device memory.  Calls enqueue
 * work on the given stream and return without waiting (except where stated).  For fixed arguments
 * the output is bitwise reproducible.
 *
 * Errors: every function that returns int returns ATTN_OK (0) or a negative attn_status;
 * attn_last_error() then holds a description (per host thread).
 */
#ifndef SAWTOOTH_ATTN_H
#define SAWTOOTH_ATTN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ATTN_OK = 0,
    ATTN_ERR_INVALID_ARG = -1,    /* null pointer, non-positive size, unknown enum, bad scale, bad option */
    ATTN_ERR_UNSUPPORTED = -2,    /* head dimension other than 64 / 128; device is not compute capability 10.x */
    ATTN_ERR_ALIGNMENT = -3,      /* a base pointer is not 16-byte aligned */
    ATTN_ERR_NO_DEVICE = -4,      /* no usable CUDA device / driver */
    ATTN_ERR_CUDA = -5,           /* a CUDA runtime or driver call failed */
    ATTN_ERR_DEVICE_TIMEOUT = -6  /* a bounded wait inside the kernel ran out (see attn_device_status) */
} attn_status;

typedef enum { ATTN_SCAN_CYCLIC = 0, ATTN_SCAN_SAWTOOTH = 1 } attn_scan_order;
typedef enum { ATTN_F16 = 0, ATTN_BF16 = 1 } attn_dtype;
typedef enum { ATTN_TILE_FASTEST = 0, ATTN_HEAD_FASTEST = 1 } attn_digit_order;
typedef enum { ATTN_LAYOUT_BHND = 0, ATTN_LAYOUT_BNHD = 1 } attn_layout;
/*
 * How the static walk of Algorithm 2 groups work items.  With pairs, a unit of the walk is two W-row Q blocks of one
 * head which the CTA handles one after the other, the first scanned first-to-last and, in the sawtooth order, the
 * second last-to-first: the form with two Q tiles per loop trip that the paper's tile-based kernels use.
 *   ATTN_PAIR_MIRRORED  blocks (n-1-p, p) of a head with n blocks.  Under the causal mask block q scans q+1 blocks' worth
 *                       of K/V tiles, so every pair scans n+1: all units take the same time, the static walk is balanced,
 *                       the CTAs of a wave stay in step and, in the sawtooth order, read the same two K/V tiles at any time.
 *   ATTN_PAIR_ADJACENT  blocks (2p, 2p+1).
 *   ATTN_PAIR_NONE      one block per unit (Algorithm 2 as printed).
 *   ATTN_PAIR_DEFAULT   mirrored under the causal mask, none otherwise.  The dynamic schedule never pairs.
 */
typedef enum { ATTN_PAIR_DEFAULT = 0, ATTN_PAIR_NONE = 1, ATTN_PAIR_MIRRORED = 2, ATTN_PAIR_ADJACENT = 3 } attn_pairing;

/* Optional knobs; zero-initialise, then set what you need.  0 always means "library default". */
typedef struct {
    int max_ctas;     /* cap on the persistent grid (the "number of active SMs" of the paper's studies) */
    int kv_stages;    /* K/V tile slots in the shared-memory ring; default: as many as fit */
    int block_n;      /* K/V rows per tile: 64 or 128 (default 128) */
    int q_tiles;      /* 128-row Q tiles per work item: 1 or 2 (default 2, so W = 256 rows) */
    int digit_order;  /* attn_digit_order: how the linear work index maps to (batch, head, Q block) */
    int launch_mode;  /* 0: persistent grid (Algorithm 2); 1: one CTA per work item (Algorithm 3) */
    int l2_policy;    /* 0: no hint; 1: K/V loads carry an evict_last hint, Q loads evict_first */
    int host_chunks;  /* attn_fwd_host only: pieces the heads are cut into so that copies and kernels overlap (1..32; 0 = automatic) */
    float* lse;       /* optional DEVICE output [B, H, N] (fp32, 4-byte aligned), NULL for none: per query row the natural log of
                         the softmax denominator, ln sum_j exp(scale * q_i . k_j) over the keys the row may see (the quantity a
                         backward pass or a merge of partial results needs; outside the paper).  Ignored by attn_fwd_host. */
    int pairing;      /* attn_pairing: whether one trip of a CTA's loop takes one work item or a pair of them (see below) */
    int check_mode;   /* 1: the call waits for the device and returns ATTN_ERR_DEVICE_TIMEOUT itself if a bounded wait inside
                         its kernel (or an earlier one on the device) ran out; 0: asynchronous, poll attn_device_status */
    int kv_heads;     /* grouped-query attention (outside the paper): k and v hold [B, kv_heads, N, d], kv_heads divides H, and query
                         head h attends to K/V head h / (H / kv_heads).  0 = H (every query head has its own K/V head) */
    int layout;       /* attn_layout of q, k, v and o (outside the paper): ATTN_LAYOUT_BHND = [B, H, N, d] (default), ATTN_LAYOUT_BNHD =
                         [B, N, H, d], the order in which projection layers leave them.  lse stays [B, H, N]. */
    int reserved[2];
} attn_fwd_opts;

/* What a call with these arguments will launch; lets a caller predict L2 traffic. */
typedef struct {
    int block_m;        /* query rows per MMA tile (128) */
    int block_n;        /* K/V rows per tile */
    int q_tiles;        /* Q tiles per work item */
    int rows_per_item;  /* W = block_m * q_tiles */
    int items_per_head; /* ceil(N / W) */
    long long n_work;   /* B * H * items_per_head */
    int grid;           /* CTAs launched */
    int threads;        /* threads per CTA */
    int kv_stages;      /* ring slots (each holds one K tile or one V tile) */
    int smem_bytes;     /* dynamic shared memory per CTA */
    int sm_count;       /* SMs of the device the plan was made for */
    int pairing;        /* attn_pairing in force (never ATTN_PAIR_DEFAULT) */
    long long n_units;  /* units of the static walk: n_work, or B * H * ceil(items_per_head / 2) with pairs; grid = min(n_units, SMs) */
} attn_plan;

/* One work item as a CTA handles it (host-side replay of the device schedule). */
typedef struct {
    int cta;            /* blockIdx.x */
    int iteration;      /* the CTA's count of items handled so far (Algorithm 4's i_local) */
    long long k;        /* linear index of the unit the walk is at (k = cta, += grid); with pairs two entries share one k */
    int batch, head;
    int q_item;         /* index of the W-row block inside the head */
    int backward;       /* 1: K/V tiles scanned last to first */
    int n_kv;           /* tiles 0 .. n_kv-1 are scanned */
    int n_kv_q0, n_kv_q1; /* of those, the ones the first / second 128-row Q tile takes part in */
    int member;         /* 0 or 1: which item of its pair this is (0 without pairs) */
} attn_trace_entry;

/*
 * The forward pass (Eq. 1 via Algorithms 1, 2, 4).  q, k, v, o: DEVICE pointers, layout as above.
 * causal: 0 or 1.  scan_order: attn_scan_order.  dtype: attn_dtype.  stream: a cudaStream_t (NULL =
 * the default stream).  Asynchronous.  `o` is fully overwritten.
 * A device's first call also looks up the library's device symbols and raises the kernel's shared-memory limit; every
 * later call (attn_fwd_ex without check_mode and attn_fwd_dynamic likewise) only enqueues work on `stream`, so it may be
 * captured into a CUDA graph and replayed.
 */
int attn_fwd(const void* q, const void* k, const void* v, void* o,
             int B, int H, int N, int d, float scale, int causal, int scan_order,
             int dtype, void* stream);

/* Same with options (opts may be NULL). */
int attn_fwd_ex(const void* q, const void* k, const void* v, void* o,
                int B, int H, int N, int d, float scale, int causal, int scan_order,
                int dtype, void* stream, const attn_fwd_opts* opts);

/*
 * The same forward pass with a DYNAMIC tile schedule in place of Algorithm 2's static grid-stride walk (the paper's
 * persistent loop hands CTA c the items c, c+G, ...; under the causal mask those differ in length by up to the whole
 * sequence, and CTAs that drew short ones idle at the end).  Here every persistent CTA claims its next work item from
 * a counter in `scratch`, in index order, which under the causal mask runs from the longest Q block of a head to the
 * shortest.  Algorithm 4's alternation follows the round of a claim (claim index / grid size): that is the CTA's own
 * count of items as long as the CTAs stay in step, and it does not depend on which CTA won the claim, so for fixed
 * arguments the result is reproducible bit for bit in both scan orders although the assignment of items to CTAs is not
 * (without the causal mask it is the static, unpaired schedule's result).
 *
 * scratch: DEVICE memory owned by the caller, 4-byte aligned, at least attn_dynamic_scratch_bytes(plan.grid) bytes
 * (plan from attn_query_plan with opts->pairing = ATTN_PAIR_NONE, since single items are claimed here;
 * ATTN_DYNAMIC_SCRATCH_HEADER + 4 bytes per CTA; the SM count of the device is always enough).  The call clears it on `stream` before
 * the kernel; afterwards int[0] holds the number of claims made and int[64 + c] the number of items CTA c handled.
 * Two calls that share one scratch buffer must not overlap on the GPU.  launch_mode must be 0.
 */
#define ATTN_DYNAMIC_SCRATCH_HEADER 256
size_t attn_dynamic_scratch_bytes(int ctas);
int attn_fwd_dynamic(const void* q, const void* k, const void* v, void* o,
                     int B, int H, int N, int d, float scale, int causal, int scan_order,
                     int dtype, void* stream, const attn_fwd_opts* opts,
                     void* scratch, size_t scratch_bytes);

/*
 * attn_fwd_dynamic for callers that cannot hand over scratch memory.  (The paper has no counterpart: this is a
 * packaging of the dynamic schedule, not a step of the method.)
 *
 * Who needs it: code that runs where device allocation is off the table -- inside a region that is being recorded
 * for replay, inside a framework's allocator callback, in a real-time loop with a no-allocation rule, or in a plug-in
 * whose host application owns all device memory.  Such a caller has nowhere to get the counter buffer from, so here
 * the buffer is a fixed array inside the library's own device image: ATTN_DYNAMIC_SCRATCH_HEADER + 4 *
 * ATTN_NOALLOC_MAX_CTAS bytes (4352), present on every GPU the library is loaded on until the process exits.
 * The call allocates and frees nothing; q, k, v, o are the caller's as everywhere else.
 *
 * Limits and rules.  A launch of more than ATTN_NOALLOC_MAX_CTAS persistent CTAs (grid of attn_query_plan) is
 * refused with ATTN_ERR_INVALID_ARG before anything is enqueued.  The first call on each device looks up the
 * array's address on that device (the device must be current); make that first call outside any stream capture.
 * All calls on one device share the one array: it still holds the previous call's counters, every call clears them
 * on `stream` before its kernel, and two calls that may run on the GPU at the same time (different streams) race
 * on it -- serialise them, or use attn_fwd_dynamic with a buffer per stream.  Device indices up to 63.
 */
#define ATTN_NOALLOC_MAX_CTAS 1024
int attn_fwd_dynamic_noalloc(const void* q, const void* k, const void* v, void* o,
                             int B, int H, int N, int d, float scale, int causal, int scan_order,
                             int dtype, void* stream, const attn_fwd_opts* opts);

/*
 * Same computation for HOST buffers: copies q, k, v (host, pinned if the copies are to overlap anything) into the
 * caller's device staging buffers q_dev, k_dev, v_dev, runs attn_fwd_ex into o_dev and copies o_dev back to o_host.
 * Each buffer holds B*H*N*d 16-bit elements.  The heads are independent, so the work is cut into opts->host_chunks
 * equal groups of heads; left to the library (0), one group per 16 MiB of a tensor once a tensor exceeds 32 MiB, 32
 * at most and a head at least (attn_host_groups tells which): upload and kernel take about as long as each other on a
 * PCIe 5 link, so the first kernel should start early and none should wait for a long upload.  The groups run as a
 * pipeline on streams the library keeps per device: upload of group i+1, kernel of group i and download of group i-1
 * proceed together, and the kernels of successive groups alternate between two streams, so that the CTAs of group i+1
 * move onto the SMs that the last round of group i leaves idle.  The
 * pipeline starts after everything already enqueued on `stream` and `stream` waits for its end, so to the caller it
 * behaves like work enqueued on `stream`.  Returns without waiting: o_host is valid once `stream` has been
 * synchronised.  The first pipelined call on a device creates the streams and events (no device memory).
 * Every argument and option is checked before the first copy is enqueued; if a CUDA call fails later, `stream` is still
 * made to wait for whatever the side streams were given.  The per-device pipeline is shared: calls from several host
 * threads (or on several caller streams) are enqueued one after the other under a lock and their pipelines run one
 * after the other on the side streams.  opts->lse is ignored, opts->check_mode must be 0.
 */
int attn_fwd_host(const void* q_host, const void* k_host, const void* v_host, void* o_host,
                  void* q_dev, void* k_dev, void* v_dev, void* o_dev,
                  int B, int H, int N, int d, float scale, int causal, int scan_order,
                  int dtype, void* stream, const attn_fwd_opts* opts);

/*
 * Host-only: the groups of heads attn_fwd_host cuts B*H = `heads` heads of `head_bytes` bytes each into, for
 * opts->host_chunks = host_chunks.  Writes the group sizes, in order, to sizes[0 .. *n - 1]; `sizes` holds at least 32
 * entries.  They sum to `heads`.  The paper has no counterpart: it times kernels on resident tensors.
 */
int attn_host_groups(long long heads, size_t head_bytes, int host_chunks, long long* sizes, int* n);

/*
 * The launch plan for these arguments (Algorithm 2's grid size, the tile shapes).  sm_count <= 0
 * means "ask the current device" (fails with ATTN_ERR_NO_DEVICE without one).
 */
int attn_query_plan(int B, int H, int N, int d, int causal, int dtype,
                    const attn_fwd_opts* opts, int sm_count, attn_plan* out);

/*
 * Host-only replay of the schedule (Algorithms 2 and 4 plus the causal tile ranges): writes up to
 * `cap` entries, CTA by CTA, each CTA's items in the order it handles them, and the total number of
 * entries to *n.  Needs no device when sm_count > 0.
 */
int attn_schedule_trace(int B, int H, int N, int d, int causal, int scan_order, int dtype,
                        const attn_fwd_opts* opts, int sm_count,
                        attn_trace_entry* buf, size_t cap, size_t* n);

/*
 * Host-only replay of the dynamic schedule (attn_fwd_dynamic): the work items in the order in which they are claimed,
 * each with the scan direction that the round of its claim gives it.  Which CTA takes a claim is not determined:
 * entries carry cta = -1, iteration = the round (claim index / grid size), k = the claim index, member = 0.
 * Arguments as for attn_schedule_trace; opts->pairing is ignored.
 */
int attn_dynamic_claim_trace(int B, int H, int N, int d, int causal, int scan_order, int dtype,
                             const attn_fwd_opts* opts, int sm_count,
                             attn_trace_entry* buf, size_t cap, size_t* n);

/*
 * Waits for the current device and reads, then clears, its kernel status word: 0, or a code naming
 * the wait that ran out in a kernel launched since the last call.  Returns ATTN_OK when the word
 * was 0, ATTN_ERR_DEVICE_TIMEOUT otherwise (code in *code if code != NULL).
 */
int attn_device_status(int* code);

/*
 * Waits for the current device and returns the SM clock cycles that the first CTA of the most recent
 * attention kernel spent in its loop over work items (a measuring aid: cycles / elapsed time is the
 * SM clock the kernel really ran at, which on a power-capped GPU is not the nominal one).
 */
int attn_last_kernel_cycles(unsigned long long* cycles);

const char* attn_status_string(int status);
const char* attn_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SAWTOOTH_ATTN_H */
