// FlashAttention forward kernel for sm_100a: persistent CTAs, TMA-fed K/V ring, tcgen05 MMAs with
// S, P and O in tensor memory, one softmax thread per query row, O written by TMA stores.
//
// One CTA handles work items of kQTiles x 128 query rows (Algorithm 1's resident Q tile).  Warp roles:
//   eight softmax warps    two threads per query row: warps w and w + 4 own TMEM lanes 32 (w % 4) .. + 31,
//                          the first the lower half of a tile's key columns (and of O's columns), the
//                          second the upper half.  All eight work on the SAME Q tile at a time and take
//                          the tiles of a work item in turn, K/V step by K/V step: while they run the
//                          softmax of one tile the tensor core runs the other tile's products, and one
//                          tile's softmax has the whole SM's exponential throughput and issue slots, which
//                          halves the latency between a tile's S and its P.  A thread reads its half of S
//                          from TMEM, swaps its partial row maximum with its partner through shared memory
//                          (an mbarrier per warp pair), keeps the running max and a partial sum, writes P
//                          back over its own S columns as 16-bit pairs in two parts, rescales its half of
//                          O when the max moved, and at the end of the item normalises its half of the O
//                          row and stages it in shared memory, from where one lane per warp issues a TMA
//                          store.
//   the next warp          producer: one elected lane issues the TMA loads (Q tiles, then K_j, V_j in
//                          the scan order of the item, then one empty slot: the item's O staging buffer)
//                          into a ring of shared-memory slots.
//   the next kQTiles warps MMA, one warp per Q tile q: one elected lane issues S_q = Q_q K_j^T and
//                          O_q += P_q V_j and commits them to mbarriers; the first of them also owns
//                          the TMEM allocation.
//   the remaining warp(s)  idle; they complete the warpgroup whose registers go to the softmax threads.
// Work items come from Algorithm 2's grid-stride walk or, with a counter in global memory, are claimed
// dynamically; Algorithm 4's scan direction follows the CTA's own item count either way.
#pragma once
#include "ptx.cuh"
#include "schedule.h"

namespace sawtooth {

// Optional in-kernel clock stamps (build with -DSAW_PROFILE): one thread of each role of every CTA adds up
// the SM cycles it spends in each phase; the host reads the table with attn_debug_profile().
#ifdef SAW_PROFILE
__device__ unsigned long long g_profile[256][32];
#define SAW_PROF_DECL long long prof_t = clock64(); long long prof_acc[12] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}
#define SAW_PROF(slot) do { const long long prof_n = clock64(); prof_acc[slot] += prof_n - prof_t; prof_t = prof_n; } while (0)
#define SAW_PROF_WRITE(base, cond) do { if (cond) { for (int prof_i = 0; prof_i < 12; ++prof_i) g_profile[blockIdx.x & 255][(base) + prof_i] = (unsigned long long)prof_acc[prof_i]; } } while (0)
#else
#define SAW_PROF_DECL do { } while (0)
#define SAW_PROF(slot) do { } while (0)
#define SAW_PROF_WRITE(base, cond) do { } while (0)
#endif

struct KernelParams {
    SchedParams sched;
    float scale_log2;     // scale * log2(e): probabilities are computed with ex2
    int kv_stages;        // slots in the K/V ring
    int l2_policy;        // 1: K/V loads evict_last, Q loads evict_first
    void* o;              // [B, H, N, d] output
    int* status;          // device status word (0 = fine)
    unsigned long long* cycles;  // CTA 0 leaves the SM cycles its MMA loop took here
    int* work_counter;    // dynamic schedule: [0] next unclaimed work index (zero at launch), [64 + cta] items the CTA
                          // handled; nullptr: the static grid-stride schedule of Algorithm 2
};

constexpr int kMaxStages = 16;
#ifndef SAW_EXP_POLY_OF_4
#define SAW_EXP_POLY_OF_4 1
#endif
constexpr int kExpPolyOf4 = SAW_EXP_POLY_OF_4;  // of every four pairs of exponentials, how many avoid the MUFU
constexpr float kRescaleThreshold = 8.0f;  // O and l are rescaled only when the row max grew by more (log2 units)

// Codes written to the status word: which wait gave up.
enum WaitSite {
    kSiteProducerQ = 1, kSiteProducerKV = 2, kSiteMmaQ = 3, kSiteMmaKV = 4, kSiteMmaP = 5,
    kSiteSoftmaxS = 6, kSiteSoftmaxO = 7, kSiteSmemAlignment = 8, kSiteWorkFull = 9, kSiteWorkEmpty = 10,
    kSiteStageSlot = 11, kSiteStageDone = 12, kSiteExchange = 13
};

struct __align__(8) Barriers {
    uint64_t q_full, q_empty;
    uint64_t kv_full[kMaxStages], kv_empty[kMaxStages];
    uint64_t s_full[2], p_early[2], p_full[2], o_full[2];
    uint64_t drain[2];
    uint64_t stage_done;                    // staged epilogue: the eight softmax warps have read their staging buffers out
    uint64_t pair[4];                       // per pair of softmax warps (w, w + 4): both have published their partial row value
    uint64_t work_full[2], work_empty[2];  // dynamic schedule: two-slot mailbox of claimed work indices
    long long work_k[2];
    uint32_t tmem_base;
    int abort_flag;
    float xchg[2][2][128];  // [exchange count & 1][column half][row]: the partial row maximum (or, at the end of an item,
                            // the partial row sum) each thread of a row shows its partner
};

template <int kD, int kBlockN, int kQTiles>
struct Geometry {
    static constexpr int kChunks = kD / 64;                 // 64-element (128-byte) column blocks per row
    static constexpr int kQTileBytes = kBlockM * kD * 2;
    static constexpr int kKVTileBytes = kBlockN * kD * 2;
    static constexpr int kQChunkBytes = kBlockM * 128;
    static constexpr int kKVChunkBytes = kBlockN * 128;
    static constexpr int kColsS = kBlockN / 2;              // S columns a softmax thread owns (two threads per row)
    static constexpr int kColsO = kD / 2;                   // O columns a softmax thread owns
    // P reaches the MMA warp in two parts: a thread announces its first kEarlyGroups groups of 16
    // probabilities (one K step of the P.V product each) while it still computes the rest.  A thread writes its
    // P over the first half of its own S columns, so the 16 keys of K step kk of the P.V product sit at column
    // (kk / kGroups) * kColsS + (kk % kGroups) * 8 of the tile's S block.
    static constexpr int kGroups = kColsS / 16;
    static constexpr int kEarlyGroups = kGroups >= 4 ? (kGroups * 3) / 4 : kGroups / 2;
    static constexpr int kSoftmaxWarps = 8;
    static constexpr int kSoftmaxThreads = kSoftmaxWarps * 32;
    static constexpr int kThreads = kSoftmaxThreads + 128;  // plus one warpgroup: producer, MMA warps, idle warp(s)
    // Epilogue through shared memory: after the last V tile of a work item the ring holds one more slot that
    // nothing is loaded into.  Each softmax warp owns an eighth of it and stages there, one Q tile after the other,
    // kStageRows rows of its kColsO 16-bit O columns at a time, written out by TMA stores (rows beyond N are
    // dropped by the copy engine).
    static constexpr int kStageBytesPerWarp = kKVTileBytes / kSoftmaxWarps;
    static constexpr int kStageRowBytes = kColsO * 2;       // 128 (d = 128) or 64 (d = 64)
    static constexpr int kStageRows = kStageBytesPerWarp / kStageRowBytes < 32 ? kStageBytesPerWarp / kStageRowBytes : 32;
    // Registers: the launch gives each of the 384 threads 65536 / 384 rounded down to a multiple of 8 = 168; the last
    // warpgroup hands registers back and the softmax warpgroups take them (256 * 200 + 128 * 104 = 384 * 168).
    static constexpr int kRegsOther = 104;
    static constexpr int kRegsSoftmax = 200;
    static constexpr int kTmemCols = 512;
    static constexpr int kTmemS = 0;      // S_q (fp32, kBlockN columns) at kTmemS + 128 q; P_q overwrites parts of it
    static constexpr int kTmemO = 256;    // O_q (fp32, kD columns) at kTmemO + 128 q
    static constexpr size_t smem_bytes(int stages) {
        return (size_t)kQTiles * kQTileBytes + (size_t)stages * kKVTileBytes + sizeof(Barriers);
    }
};

struct Ring {
    int slot = 0;
    uint32_t phase = 0;
    __device__ __forceinline__ void advance(int stages) {
        if (++slot == stages) { slot = 0; phase ^= 1u; }
    }
    __device__ __forceinline__ void advance_by(int n, int stages) {
        const int t = slot + n;
        slot = t % stages;
        phase ^= (uint32_t)(t / stages) & 1u;
    }
};

// Short wait that ignores the abort flag: used on the way out, for copies and MMAs still in flight.
__device__ __forceinline__ void drain_wait(uint64_t* bar, uint32_t parity) {
    const unsigned long long t0 = ptx::global_ns();
    while (!ptx::mbar_try_wait(bar, parity)) {
        if (ptx::global_ns() - t0 > 2000000ull) break;
    }
}

template <int kD, int kBlockN, int kQTiles, int kBf16>
__global__ void __launch_bounds__(Geometry<kD, kBlockN, kQTiles>::kThreads, 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o, const KernelParams p)
{
    using G = Geometry<kD, kBlockN, kQTiles>;
    extern __shared__ __align__(1024) uint8_t smem[];
    if ((ptx::smem_u32(smem) & 1023u) != 0) {  // the swizzled tiles need a 1024-byte aligned base
        if (threadIdx.x == 0) atomicCAS(p.status, 0, (int)kSiteSmemAlignment);
        return;
    }
    uint8_t* q_smem = smem;
    uint8_t* kv_smem = smem + kQTiles * G::kQTileBytes;
    Barriers* bar = reinterpret_cast<Barriers*>(kv_smem + (size_t)p.kv_stages * G::kKVTileBytes);
    volatile int* abort_flag = &bar->abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    constexpr int kProducerWarp = G::kSoftmaxWarps;
    constexpr int kMmaWarp = G::kSoftmaxWarps + 1;
    const int stages = p.kv_stages;

    if (tid == 0) {
        ptx::mbar_init(&bar->q_full, 1);
        ptx::mbar_init(&bar->q_empty, kQTiles);
        for (int s = 0; s < stages; ++s) {
            ptx::mbar_init(&bar->kv_full[s], 1);
            ptx::mbar_init(&bar->kv_empty[s], kQTiles);
        }
        for (int q = 0; q < 2; ++q) {
            ptx::mbar_init(&bar->s_full[q], 1);
            ptx::mbar_init(&bar->p_early[q], G::kSoftmaxWarps);
            ptx::mbar_init(&bar->p_full[q], G::kSoftmaxWarps);
            ptx::mbar_init(&bar->o_full[q], 1);
        }
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(&bar->work_full[i], 1);
            ptx::mbar_init(&bar->work_empty[i], kQTiles + G::kSoftmaxWarps);
        }
        for (int i = 0; i < 4; ++i) ptx::mbar_init(&bar->pair[i], 2);
        ptx::mbar_init(&bar->stage_done, G::kSoftmaxWarps);
        ptx::mbar_init(&bar->drain[0], 1);
        ptx::mbar_init(&bar->drain[1], 1);
        bar->abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == kProducerWarp && lane == 0) {
        ptx::prefetch_tmap(&tm_q);
        ptx::prefetch_tmap(&tm_k);
        ptx::prefetch_tmap(&tm_v);
        ptx::prefetch_tmap(&tm_o);
    }
    if (warp == kMmaWarp) {
        ptx::tmem_alloc(&bar->tmem_base, G::kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = bar->tmem_base;

    // Which work item this CTA handles as its iteration `it` (-1: none left).  Static schedule (Algorithm 2):
    // blockIdx.x + it * gridDim.x.  Dynamic schedule: the producer warp claims the next unclaimed index from a
    // global counter and passes it to the other roles through a two-slot mailbox in shared memory, so a CTA
    // that drew short items simply draws more of them; Algorithm 4's parity stays the CTA's own count `it`.
    const bool dynamic = p.work_counter != nullptr;
    auto static_work = [&](int it) -> long long {
        const long long k = (long long)blockIdx.x + (long long)it * gridDim.x;
        return k < p.sched.n_work ? k : -1;
    };
    auto claim_work = [&](int it, bool& ok) -> long long {  // producer warp, all lanes
        if (!dynamic) return static_work(it);
        const int slot = it & 1;
        if (it >= 2) {
            ok = ptx::warp_all(ptx::mbar_wait(&bar->work_empty[slot], (uint32_t)(((it >> 1) & 1) ^ 1), abort_flag, kSiteWorkEmpty));
            if (!ok) return -1;
        }
        if (ptx::elect_one()) {
            const long long c = (long long)atomicAdd(p.work_counter, 1);
            bar->work_k[slot] = c < p.sched.n_work ? c : -1;
            ptx::mbar_arrive(&bar->work_full[slot]);
        }
        __syncwarp();
        return bar->work_k[slot];
    };
    auto take_work = [&](int it, bool& ok, bool whole_warp) -> long long {  // MMA lanes (one thread), softmax warps
        if (!dynamic) return static_work(it);
        const int slot = it & 1;
        if (!ptx::mbar_wait(&bar->work_full[slot], (uint32_t)((it >> 1) & 1), abort_flag, kSiteWorkFull)) { ok = false; return -1; }
        const long long k = bar->work_k[slot];
        if (whole_warp) {
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&bar->work_empty[slot]);
        } else {
            ptx::mbar_arrive(&bar->work_empty[slot]);
        }
        return k;
    };

    if (warp >= G::kSoftmaxWarps) {
    // The last warpgroup (producer, MMA and idle warps) hands registers back in one instruction.  (Its three
    // roles below keep the indentation of the outer level.)
    ptx::reg_dealloc<G::kRegsOther>();
    if (warp == kProducerWarp) {
        // ------------------------------------------------------------------ producer
        // The whole warp walks the schedule and waits on the barriers; one elected lane issues the
        // copies (elect.sync keeps the issue path warp-uniform for the compiler).
        uint64_t pol_kv = 0, pol_q = 0;
        if (p.l2_policy) { pol_kv = ptx::policy_evict_last(); pol_q = ptx::policy_evict_first(); }
        Ring ring;
        uint32_t q_issued = 0;     // Q loads issued so far
        long long kv_issued = 0;   // K/V tile loads issued so far
        bool ok = true;
        int it = 0;
        for (; ok; ++it) {
            const long long k = claim_work(it, ok);
            if (!ok || k < 0) break;
            const WorkItem w = decode_work(p.sched, k, it);
            ok = ptx::warp_all(ptx::mbar_wait(&bar->q_empty, (it & 1) ^ 1, abort_flag, kSiteProducerQ));
            if (!ok) break;
            if (ptx::elect_one()) {
                int n_valid = 0;
#pragma unroll
                for (int q = 0; q < kQTiles; ++q) n_valid += (w.hi_q[q] > 0);
                ptx::mbar_arrive_expect_tx(&bar->q_full, (uint32_t)n_valid * G::kQTileBytes);
#pragma unroll
                for (int q = 0; q < kQTiles; ++q) {
                    if (w.hi_q[q] == 0) continue;
#pragma unroll
                    for (int c = 0; c < G::kChunks; ++c) {
                        void* dst = q_smem + q * G::kQTileBytes + c * G::kQChunkBytes;
                        if (p.l2_policy) ptx::tma_load_3d_hint(dst, &tm_q, &bar->q_full, c * 64, w.row0 + q * kBlockM, w.bh, pol_q);
                        else ptx::tma_load_3d(dst, &tm_q, &bar->q_full, c * 64, w.row0 + q * kBlockM, w.bh);
                    }
                }
            }
            __syncwarp();
            ++q_issued;
            for (int s = 0; ok && s < w.hi; ++s) {
                const int j = kv_tile_at(w, s);
                for (int kv = 0; kv < 2; ++kv) {
                    ok = ptx::warp_all(ptx::mbar_wait(&bar->kv_empty[ring.slot], ring.phase ^ 1u, abort_flag, kSiteProducerKV));
                    if (!ok) break;
                    if (ptx::elect_one()) {
                        ptx::mbar_arrive_expect_tx(&bar->kv_full[ring.slot], G::kKVTileBytes);
                        const CUtensorMap* tm = kv ? &tm_v : &tm_k;
#pragma unroll
                        for (int c = 0; c < G::kChunks; ++c) {
                            void* dst = kv_smem + (size_t)ring.slot * G::kKVTileBytes + c * G::kKVChunkBytes;
                            if (p.l2_policy) ptx::tma_load_3d_hint(dst, tm, &bar->kv_full[ring.slot], c * 64, j * kBlockN, w.bh, pol_kv);
                            else ptx::tma_load_3d(dst, tm, &bar->kv_full[ring.slot], c * 64, j * kBlockN, w.bh);
                        }
                    }
                    __syncwarp();
                    ring.advance(stages);
                    ++kv_issued;
                }
            }
            if (ok) {
                // The item's staging slot: wait until its last contents are consumed, then hand it to the softmax warps
                // through the slot's own full barrier (no bytes are expected).
                ok = ptx::warp_all(ptx::mbar_wait(&bar->kv_empty[ring.slot], ring.phase ^ 1u, abort_flag, kSiteProducerKV));
                if (!ok) break;
                if (ptx::elect_one()) ptx::mbar_arrive(&bar->kv_full[ring.slot]);
                __syncwarp();
                ring.advance(stages);
                ++kv_issued;
            }
        }
        if (dynamic && lane == 0) p.work_counter[64 + blockIdx.x] = it;
        if (!ok) {
            // Leave no copy in flight: wait (briefly) for the loads issued last into each slot.
            if (q_issued) drain_wait(&bar->q_full, (q_issued - 1) & 1u);
            const int back = kv_issued < stages ? (int)kv_issued : stages;
            Ring r = ring;
            for (int n = 0; n < back; ++n) {
                if (r.slot == 0) { r.slot = stages - 1; r.phase ^= 1u; } else { --r.slot; }
                drain_wait(&bar->kv_full[r.slot], r.phase);
            }
        }
        __syncwarp();
    } else if (warp < kMmaWarp + kQTiles) {
        // ------------------------------------------------------------------ MMA issue
        // One warp per Q tile, one elected lane each: the products of the two tiles are independent, so
        // a lane that waits for its tile's P does not hold up the other tile's products.  Both lanes walk
        // the same K/V ring; a slot, and the Q buffer, are free again once both have committed.
        const int q = warp - kMmaWarp;
        constexpr uint32_t idesc_qk = ptx::instr_desc_f16(kBf16, 0, kBlockM, kBlockN);
        constexpr uint32_t idesc_pv = ptx::instr_desc_f16(kBf16, 1, kBlockM, kD);
        const uint32_t q_base = ptx::smem_u32(q_smem);
        const uint32_t kv_base = ptx::smem_u32(kv_smem);
        Ring ring;
        uint32_t p_phase = 0;
        bool ok = true;

        // Descriptors differ from a base only in the 16-byte-granular address field (the low bits).
        const uint64_t q_desc = ptx::smem_desc_sw128(q_base, 16, 1024) + (uint64_t)((q * G::kQTileBytes) >> 4);
        const uint64_t k_desc0 = ptx::smem_desc_sw128(kv_base, 16, 1024);
        const uint64_t v_desc0 = ptx::smem_desc_sw128(kv_base, G::kKVChunkBytes, 1024);
        const uint32_t s_tmem = tmem + G::kTmemS + 128 * q;
        const uint32_t o_tmem = tmem + G::kTmemO + 128 * q;
        auto issue_qk = [&](int slot) {
            const uint64_t b0 = k_desc0 + (uint64_t)((slot * G::kKVTileBytes) >> 4);
#pragma unroll
            for (int i = 0; i < G::kChunks * 4; ++i) {
                const int c = i >> 2, kk = i & 3;
                ptx::mma_ss(s_tmem, q_desc + (uint64_t)((c * G::kQChunkBytes + kk * 32) >> 4),
                            b0 + (uint64_t)((c * G::kKVChunkBytes + kk * 32) >> 4), idesc_qk, i != 0);
            }
        };
        // The K steps of O_q += P_q V_j whose 16 probabilities belong to the early part of P (late = 0) or
        // to the rest (late = 1); a sum, so the order of the steps is free.
        auto issue_pv = [&](int slot, uint32_t accumulate, int late) {
            const uint64_t b0 = v_desc0 + (uint64_t)((slot * G::kKVTileBytes) >> 4);
#pragma unroll
            for (int kk = 0; kk < kBlockN / 16; ++kk) {
                if (((kk % G::kGroups) >= G::kEarlyGroups) != (late != 0)) continue;
                ptx::mma_ts(o_tmem, s_tmem + (kk / G::kGroups) * G::kColsS + (kk % G::kGroups) * 8,
                            b0 + (uint64_t)(kk * ((16 * 128) >> 4)), idesc_pv, accumulate | (late != 0) | (kk != 0));
            }
        };

        // The elected lane runs the whole loop: every wait, issue and commit below is a single
        // thread's, with no warp votes or re-convergence between the MMA batches.
        if (ptx::elect_one()) {
            const long long clk_begin = clock64();
            SAW_PROF_DECL;
            int it = 0;
            for (; ok; ++it) {
                const long long k = take_work(it, ok, false);
                if (!ok || k < 0) break;
                const WorkItem w = decode_work(p.sched, k, it);
                const int hi_mine = q ? w.hi_q[1] : w.hi_q[0];
                SAW_PROF(0);
                if (!ptx::mbar_wait(&bar->q_full, it & 1, abort_flag, kSiteMmaQ)) { ok = false; break; }
                SAW_PROF(1);
                // K tile of step 0
                const int slot_k = ring.slot;
                if (!ptx::mbar_wait(&bar->kv_full[slot_k], ring.phase, abort_flag, kSiteMmaKV)) { ok = false; break; }
                ring.advance(stages);
                ptx::tc_fence_after();
                if (kv_tile_at(w, 0) < hi_mine) { issue_qk(slot_k); ptx::mma_commit(&bar->s_full[q]); }
                ptx::mma_commit(&bar->kv_empty[slot_k]);
                if (w.hi == 1) ptx::mma_commit(&bar->q_empty);
                uint32_t pv_started = 0;
                for (int s = 0; ok && s < w.hi; ++s) {
                    const int j = kv_tile_at(w, s);
                    const bool has_next = s + 1 < w.hi;
                    const int j_next = has_next ? kv_tile_at(w, s + 1) : 0;
                    const int slot_v = ring.slot;
                    SAW_PROF(0);
                    if (!ptx::mbar_wait(&bar->kv_full[slot_v], ring.phase, abort_flag, kSiteMmaKV)) { ok = false; break; }
                    ring.advance(stages);
                    int slot_kn = 0;
                    if (has_next) {
                        slot_kn = ring.slot;
                        if (!ptx::mbar_wait(&bar->kv_full[slot_kn], ring.phase, abort_flag, kSiteMmaKV)) { ok = false; break; }
                        ring.advance(stages);
                    }
                    SAW_PROF(2);
                    if (j < hi_mine) {
                        if (!ptx::mbar_wait(&bar->p_early[q], p_phase, abort_flag, kSiteMmaP)) { ok = false; break; }
                        SAW_PROF(3);
                        ptx::tc_fence_after();
                        issue_pv(slot_v, pv_started, 0);
                        SAW_PROF(4);
                        if (!ptx::mbar_wait(&bar->p_full[q], p_phase, abort_flag, kSiteMmaP)) { ok = false; break; }
                        SAW_PROF(5);
                        p_phase ^= 1u;
                        ptx::tc_fence_after();
                        issue_pv(slot_v, pv_started, 1);
                        pv_started = 1;
                        SAW_PROF(6);
                    }
                    if (has_next && j_next < hi_mine) {
                        ptx::tc_fence_after();
                        issue_qk(slot_kn);
                        ptx::mma_commit(&bar->s_full[q]);
                        SAW_PROF(7);
                    }
                    // Every lane commits every slot, used by its tile or not: the slot's count is the number of lanes.
                    ptx::mma_commit(&bar->kv_empty[slot_v]);
                    if (has_next) {
                        ptx::mma_commit(&bar->kv_empty[slot_kn]);
                        if (s + 2 == w.hi) ptx::mma_commit(&bar->q_empty);  // the item's last S product is issued
                    }
                    SAW_PROF(8);
                }
                if (!ok) break;
                if (hi_mine > 0) ptx::mma_commit(&bar->o_full[q]);
                // The staging slot is released by the softmax warps on behalf of every tile they stored, and here for a
                // tile that lies beyond N.
                if (hi_mine == 0) ptx::mbar_arrive(&bar->kv_empty[ring.slot]);
                ring.advance(stages);
            }
            // Nothing of this thread's MMAs may be in flight when TMEM is released.
            ptx::mma_commit(&bar->drain[q]);
            drain_wait(&bar->drain[q], 0);
            if (blockIdx.x == 0 && q == 0) *p.cycles = (unsigned long long)(clock64() - clk_begin);
            SAW_PROF_WRITE(0, q == 0);
        }
        __syncwarp();
    }
    } else {
        // ------------------------------------------------------------------ softmax / correction / epilogue
        ptx::reg_alloc<G::kRegsSoftmax>();
        constexpr int kColsS = G::kColsS, kColsO = G::kColsO;
        const int half = warp >> 2;                    // which half of a row's key columns and of its O columns
        const int wq = warp & 3;                       // which quarter of the tile's rows = of the TMEM lanes
        const int r_in_tile = wq * 32 + lane;          // row inside a tile = TMEM lane
        const uint32_t lane_base = (uint32_t)(wq * 32) << 16;
        const uint32_t t_s0 = tmem + lane_base + G::kTmemS + half * kColsS;   // + 128 q: this thread's S (and P) columns
        const uint32_t t_o0 = tmem + lane_base + G::kTmemO + half * kColsO;   // + 128 q: this thread's O columns
        uint64_t* pair_bar = &bar->pair[wq];
        const float scale_log2 = p.scale_log2;
        const int N = p.sched.N;
        uint32_t s_phases = 0, o_phases = 0;   // bit q: parity of the next phase of s_full[q] / o_full[q]
        uint32_t xcount = 0;       // exchanges with the partner thread so far (picks the buffer and the barrier phase)
        bool ok = true;
        int it = 0;
        Ring ring;                 // position of the next work item's first K tile in the K/V ring
        uint32_t stage_phase = 0;
        SAW_PROF_DECL;
        // The two threads of a row show each other a partial value (row maximum, row sum) through shared memory: show()
        // publishes this thread's, partner() waits for the other's.  Successive exchanges alternate between two buffers.
        auto show = [&](float mine) {
            bar->xchg[xcount & 1][half][r_in_tile] = mine;
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(pair_bar);
        };
        auto partner = [&](float& theirs) -> bool {
            const bool got = ptx::mbar_wait(pair_bar, xcount & 1u, abort_flag, kSiteExchange);
            theirs = bar->xchg[xcount & 1][half ^ 1][r_in_tile];
            ++xcount;
            return got;
        };
        for (; ok; ++it) {
            const long long k = take_work(it, ok, true);
            if (!ok || k < 0) break;
            const WorkItem w = decode_work(p.sched, k, it);
            ring.advance_by(2 * w.hi, stages);   // now at the item's staging slot
            const Ring stage = ring;
            ring.advance(stages);
            // Running max (the reference the exponents are taken against, log2 units) and this thread's partial sum
            // of probabilities, for the tile handled now (_a) and for the other one (_b).
            float m_a = -INFINITY, l_a = 0.f, m_b = -INFINITY, l_b = 0.f;
            bool first_a = true, first_b = true;
            for (int s = 0; ok && s < w.hi; ++s) {
                const int j = kv_tile_at(w, s);
#pragma unroll 1
                for (int q = 0; q < kQTiles; ++q) {
                    const int hi_mine = q ? w.hi_q[1] : w.hi_q[0];
                    if (j < hi_mine) {
                        const int tile_row0 = w.row0 + q * kBlockM;
                        const int row = tile_row0 + r_in_tile;
                        const uint32_t t_s = t_s0 + 128 * q, t_o = t_o0 + 128 * q;
                        SAW_PROF(0);
                        const bool got_s = ptx::mbar_wait(&bar->s_full[q], (s_phases >> q) & 1u, abort_flag, kSiteSoftmaxS);
                        s_phases ^= 1u << q;
                        ptx::tc_fence_after();
                        SAW_PROF(1);

                        uint32_t sv[kColsS / 32][32];
#pragma unroll
                        for (int c = 0; c < kColsS / 32; ++c) ptx::tmem_ld32(t_s + c * 32, sv[c]);
                        ptx::tmem_wait_ld();
                        SAW_PROF(2);

                        const int col0 = j * kBlockN + half * kColsS;  // key index of this thread's first column
                        const bool masked = (j * kBlockN + kBlockN > N) || (p.sched.causal && (j * kBlockN + kBlockN - 1 > tile_row0));
                        if (masked) {
                            const int limit = p.sched.causal ? (row < N - 1 ? row : N - 1) : N - 1;  // last visible key
#pragma unroll
                            for (int c = 0; c < kColsS / 32; ++c)
#pragma unroll
                                for (int i = 0; i < 32; ++i)
                                    if (col0 + c * 32 + i > limit) sv[c][i] = 0xff800000u;  // -inf
                        }

                        // Eight independent chains of three-input maxima, then a tree.
                        float mx[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) mx[i] = ptx::max3(__uint_as_float(sv[0][3 * i]), __uint_as_float(sv[0][3 * i + 1]), __uint_as_float(sv[0][3 * i + 2]));
#pragma unroll
                        for (int i = 0; i < 4; ++i) mx[i] = ptx::max3(mx[i], __uint_as_float(sv[0][24 + 2 * i]), __uint_as_float(sv[0][25 + 2 * i]));
#pragma unroll
                        for (int c = 1; c < kColsS / 32; ++c)
#pragma unroll
                            for (int i = 0; i < 32; i += 2)
                                mx[(i >> 1) & 7] = ptx::max3(mx[(i >> 1) & 7], __uint_as_float(sv[c][i]), __uint_as_float(sv[c][i + 1]));
                        float row_max = fmaxf(ptx::max3(mx[0], mx[1], mx[2]), fmaxf(ptx::max3(mx[3], mx[4], mx[5]), fmaxf(mx[6], mx[7])));
                        // The two threads of a row swap their maxima.  (Both have loaded their S columns by now and each
                        // writes P over its own columns only, so neither can overwrite what the other still has to read.)
                        show(row_max);
                        const ptx::f32x2 scale2 = ptx::pack_f32x2(scale_log2, scale_log2);
                        ptx::f32x2 l01 = ptx::pack_f32x2(0.f, 0.f), l23 = ptx::pack_f32x2(0.f, 0.f);
                        // Groups of 16 probabilities (eight packed registers, one TMEM store each): x = S * scale * log2(e) - m
                        // as packed FMAs, then 2^x on the MUFU or, for kExpPolyOf4 of every four pairs, on the FMA pipe.
                        uint32_t pk[G::kGroups][8];
                        auto exp_group = [&](int g, ptx::f32x2 neg_m2) {
                            const int c = g >> 1, h = g & 1;
#pragma unroll
                            for (int i = 0; i < 16; i += 4) {
                                const ptx::f32x2 xa = ptx::fma2(ptx::pack_f32x2(__uint_as_float(sv[c][16 * h + i]), __uint_as_float(sv[c][16 * h + i + 1])), scale2, neg_m2);
                                const ptx::f32x2 xb = ptx::fma2(ptx::pack_f32x2(__uint_as_float(sv[c][16 * h + i + 2]), __uint_as_float(sv[c][16 * h + i + 3])), scale2, neg_m2);
                                float x0, x1, x2, x3, p0, p1, p2, p3;
                                ptx::unpack_f32x2(xa, x0, x1);
                                ptx::unpack_f32x2(xb, x2, x3);
                                if (((i >> 2) * 2) % 4 < kExpPolyOf4) ptx::exp2_poly_pair(x0, x1, p0, p1);
                                else { p0 = ptx::ex2(x0); p1 = ptx::ex2(x1); }
                                if (((i >> 2) * 2 + 1) % 4 < kExpPolyOf4) ptx::exp2_poly_pair(x2, x3, p2, p3);
                                else { p2 = ptx::ex2(x2); p3 = ptx::ex2(x3); }
                                l01 = ptx::add2(l01, ptx::pack_f32x2(p0, p1));
                                l23 = ptx::add2(l23, ptx::pack_f32x2(p2, p3));
                                pk[g][i / 2] = ptx::pack2<kBf16>(p0, p1);
                                pk[g][i / 2 + 1] = ptx::pack2<kBf16>(p2, p3);
                            }
                        };
                        // While the partner's maximum is on its way the first group is computed against the reference the
                        // row already has: the reference moves only when the row maximum grew by more than the threshold,
                        // which is rare after an item's first steps.  When it does move, the group is computed again.
                        float neg_m = (m_a == -INFINITY) ? 0.f : -m_a;
                        ptx::f32x2 neg_m2 = ptx::pack_f32x2(neg_m, neg_m);
                        exp_group(0, neg_m2);
                        SAW_PROF(3);
                        float other_max;
                        const bool got_x = partner(other_max);
                        ok = ptx::warp_all(got_s && got_x);
                        if (!ok) break;
                        row_max = fmaxf(row_max, other_max);
                        SAW_PROF(4);
                        const float m_cand = fmaxf(m_a, row_max * scale_log2);
                        const bool need = (m_cand - m_a) > kRescaleThreshold;
                        if (__any_sync(0xffffffffu, need)) {
                            float alpha = 1.f;
                            if (need) {
                                alpha = ptx::ex2(m_a - m_cand);  // 0 when nothing was accumulated yet
                                m_a = m_cand;
                                l_a *= alpha;
                            }
                            if (!first_a) {
                                // S_q is complete, so every product issued before it, O_q's last update included, is too.
#pragma unroll 1
                                for (int c = 0; c < kColsO / 16; ++c) {
                                    uint32_t ov[16];
                                    ptx::tmem_ld16(t_o + c * 16, ov);
                                    ptx::tmem_wait_ld();
#pragma unroll
                                    for (int i = 0; i < 16; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
                                    ptx::tmem_st16(t_o + c * 16, ov);
                                }
                            }
                            neg_m = (m_a == -INFINITY) ? 0.f : -m_a;
                            neg_m2 = ptx::pack_f32x2(neg_m, neg_m);
                            l01 = ptx::pack_f32x2(0.f, 0.f);
                            l23 = ptx::pack_f32x2(0.f, 0.f);
                            exp_group(0, neg_m2);
                        }
                        SAW_PROF(5);
                        // The store of a group is issued after the exponentials of the next group, so that it never waits
                        // in the instruction stream for MUFU results that are still in flight.
                        auto finish_group = [&](int g) {
                            ptx::tmem_st8(t_s + g * 8, pk[g]);
                            if (g == G::kEarlyGroups - 1) {
                                ptx::tmem_wait_st();
                                ptx::tc_fence_before();
                                __syncwarp();
                                if (lane == 0) ptx::mbar_arrive(&bar->p_early[q]);
                                SAW_PROF(6);
                            }
                        };
#pragma unroll
                        for (int g = 1; g < G::kGroups; ++g) {
                            exp_group(g, neg_m2);
                            finish_group(g - 1);
                        }
                        finish_group(G::kGroups - 1);
                        float l0, l1, l2, l3;
                        ptx::unpack_f32x2(l01, l0, l1);
                        ptx::unpack_f32x2(l23, l2, l3);
                        l_a += (l0 + l1) + (l2 + l3);
                        ptx::tmem_wait_st();
                        ptx::tc_fence_before();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(&bar->p_full[q]);
                        SAW_PROF(7);
                        first_a = false;
                    }
                    if (kQTiles == 2) {   // the other tile's state takes its turn
                        const float tm = m_a, tl = l_a;
                        const bool tf = first_a;
                        m_a = m_b; l_a = l_b; first_a = first_b;
                        m_b = tm; l_b = tl; first_b = tf;
                    }
                }
            }
            if (!ok) break;
            // ---- epilogue, one Q tile after the other: O_q / l -> 16 bit -> staging rows -> TMA store
            int tiles_stored = 0;
#pragma unroll 1
            for (int q = 0; q < kQTiles; ++q) {
                const int hi_mine = q ? w.hi_q[1] : w.hi_q[0];
                if (hi_mine > 0) {
                    const int tile_row0 = w.row0 + q * kBlockM;
                    const uint32_t t_o = t_o0 + 128 * q;
                    SAW_PROF(0);
                    const bool got_o = ptx::mbar_wait(&bar->o_full[q], (o_phases >> q) & 1u, abort_flag, kSiteSoftmaxO);
                    o_phases ^= 1u << q;
                    ptx::tc_fence_after();
                    SAW_PROF(9);
                    float other_sum;
                    show(l_a);
                    const bool got_x = partner(other_sum);
                    const bool got_slot = ptx::mbar_wait(&bar->kv_full[stage.slot], stage.phase, abort_flag, kSiteStageSlot);
                    ok = ptx::warp_all(got_o && got_x && got_slot);
                    if (!ok) break;
                    SAW_PROF(10);
                    const float inv_l = 1.f / (l_a + other_sum);
                    uint8_t* buf = kv_smem + (size_t)stage.slot * G::kKVTileBytes + (size_t)warp * G::kStageBytesPerWarp;
                    const int my_pass = lane / G::kStageRows, my_row = lane % G::kStageRows;
                    uint32_t pk[kColsO / 2];   // this thread's O columns of the row, 16-bit pairs
#pragma unroll
                    for (int c = 0; c < kColsO / 32; ++c) {
                        uint32_t ov[32];
                        ptx::tmem_ld32(t_o + c * 32, ov);
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; i += 2)
                            pk[c * 16 + i / 2] = ptx::pack2<kBf16>(__uint_as_float(ov[i]) * inv_l, __uint_as_float(ov[i + 1]) * inv_l);
                    }
#pragma unroll 1
                    for (int ps = 0; ps < 32 / G::kStageRows; ++ps) {
                        if (my_pass == ps) {
                            // Rows of 128 (64) bytes, eight to a 1024 (512)-byte swizzle atom: 16-byte piece i of row r sits
                            // at piece i ^ (r & 7) (i ^ ((r >> 1) & 3)).
                            uint4* dst_row = reinterpret_cast<uint4*>(buf + my_row * G::kStageRowBytes);
                            const int sw = G::kStageRowBytes == 128 ? (my_row & 7) : ((my_row >> 1) & 3);
#pragma unroll
                            for (int i = 0; i < G::kStageRowBytes / 16; ++i)
                                dst_row[i ^ sw] = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
                        }
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        const int y0 = tile_row0 + wq * 32 + ps * G::kStageRows;
                        if (y0 < N && ptx::elect_one()) {   // rows of the box beyond N are dropped by the copy
                            ptx::tma_store_3d(&tm_o, buf, half * kColsO, y0, w.bh);
                            ptx::bulk_commit_group();
                            ptx::bulk_wait_group_read0();   // the buffer may be written again
                        }
                        __syncwarp();
                    }
                    ++tiles_stored;
                    ptx::tc_fence_before();  // ordered before this thread's next arrive on p_full, which lets O_q be overwritten
                    SAW_PROF(11);
                }
                if (kQTiles == 2) {
                    const float tm = m_a, tl = l_a;
                    m_a = m_b; l_a = l_b;
                    m_b = tm; l_b = tl;
                }
            }
            if (!ok) break;
            // The slot goes back to the producer once all eight warps have read their buffers out: one arrival per tile
            // stored (the MMA lane of a tile beyond N makes that tile's).
            if (lane == 0) ptx::mbar_arrive(&bar->stage_done);
            if (warp == 0) {
                ok = ptx::warp_all(ptx::mbar_wait(&bar->stage_done, stage_phase, abort_flag, kSiteStageDone));
                if (ok && lane == 0)
                    for (int t = 0; t < tiles_stored; ++t) ptx::mbar_arrive(&bar->kv_empty[stage.slot]);
            }
            stage_phase ^= 1u;
            SAW_PROF(8);
        }
        ptx::bulk_wait_group0();   // this thread's TMA stores have landed before the CTA ends
        SAW_PROF_WRITE(12, warp == 0 && lane == 0);
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, G::kTmemCols);
    }
    if (tid == 0 && bar->abort_flag != 0) atomicCAS(p.status, 0, bar->abort_flag);
}

}  // namespace sawtooth
