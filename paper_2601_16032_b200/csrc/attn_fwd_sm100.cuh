// FlashAttention forward kernel for sm_100a: persistent CTAs, TMA-fed K/V ring, tcgen05 MMAs with
// S, P and O in tensor memory, one softmax thread per query row, O written by TMA stores.
//
// One CTA handles work items of kQTiles x 128 query rows (Algorithm 1's resident Q tile).  Warp roles:
//   the softmax warps      one warpgroup per Q tile, thread r owning row r (TMEM lane r).  A thread reads its
//                          row of S from TMEM, keeps the running max and sum, writes P back to TMEM as 16-bit
//                          pairs in two parts, rescales its row of O when the max moved, and at the end of the
//                          item normalises the O row and stages it in shared memory, from where one lane per
//                          warp issues a TMA store.
//   the next warp          producer: one elected lane issues the TMA loads (Q tiles, then K_j, V_j in
//                          the scan order of the item, then one empty slot: the item's O staging buffer)
//                          into a ring of shared-memory slots.
//   the next kQTiles warps MMA, one warp per Q tile q: one elected lane issues S_q = Q_q K_j^T and
//                          O_q += P_q V_j and commits them to mbarriers; the first of them also owns
//                          the TMEM allocation.
//   the remaining warp(s)  idle; they complete the warpgroup whose registers go to the softmax threads.
// With two Q tiles the tensor core works on one tile's products while the other tile's softmax runs.
// Where tensor memory has room for more S buffers than there are Q tiles (d = 64, or a single Q tile), the buffers
// are handed round in the order of the products, and S of a tile's next step is computed while the softmax of
// its present step still runs (Geometry::kEarlyQK).
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
    float scale_log2;     // |scale| * log2(e): probabilities are computed with ex2
    int negate;           // 1: scale < 0, the scores change sign before anything else is done with them
    int kv_heads;         // K/V heads per batch entry; query head h reads K/V head h / (H / kv_heads) (grouped-query attention)
    int kv_stages;        // slots in the K/V ring
    int l2_policy;        // 1: K/V loads evict_last, Q loads evict_first
    void* o;              // [B, H, N, d] output
    float* lse;           // [B, H, N] natural-log sum of exponentials per query row, or nullptr
    int* status;          // device status word (0 = fine)
    unsigned long long* cycles;  // CTA 0 leaves the SM cycles its MMA loop took here
    int* work_counter;    // dynamic schedule: [0] next unclaimed work index (zero at launch), [64 + cta] items the CTA
                          // handled; nullptr: the static grid-stride schedule of Algorithm 2
};

constexpr int kMaxStages = 16;
// Which of the eight pairs of exponentials of a group of 16 avoid the MUFU (bit i: pair i takes the cubic on the FMA
// pipe).  At d = 64 the step is as long as the softmax and a quarter of them off the MUFU is the measured optimum; at
// d = 128 the tensor core sets the step, the MUFU has room, and the extra instructions only cost power.
#ifndef SAW_EXP_POLY_MASK_D64
#define SAW_EXP_POLY_MASK_D64 0x11
#endif
#ifndef SAW_EXP_POLY_MASK_D128
#define SAW_EXP_POLY_MASK_D128 0x00
#endif
constexpr float kRescaleThreshold = 8.0f;  // O and l are rescaled only when the row max grew by more (log2 units)

// Codes written to the status word: which wait gave up.
enum WaitSite {
    kSiteProducerQ = 1, kSiteProducerKV = 2, kSiteMmaQ = 3, kSiteMmaKV = 4, kSiteMmaP = 5,
    kSiteSoftmaxS = 6, kSiteSoftmaxO = 7, kSiteSmemAlignment = 8, kSiteWorkFull = 9, kSiteWorkEmpty = 10,
    kSiteStageSlot = 11, kSiteStageDone = 12, kSiteMmaSFree = 13, kSiteSoftmaxPvDone = 14, kSiteMmaTurn = 15
};

struct __align__(8) Barriers {
    uint64_t q_full, q_empty;
    uint64_t kv_full[kMaxStages], kv_empty[kMaxStages];
    // Per Q tile and parity of the tile's product count k (two barriers taken in turn, phase (k >> 1) & 1, so that a
    // completion is never more than one ahead of the role that waits for it): S_q complete; the early part of P_q,
    // all of P_q written; the product P_q V complete (O_q up to date).
    uint64_t s_full[2][2], p_early[2][2], p_full[2][2], pv_done[2][2];
    // Per S buffer (shared by the tiles when there are more buffers than tiles): the P.V product that read its P has
    // completed.  Its waiters, the two MMA lanes, take turns in the order of the products (qk_turn), so that each use of
    // a buffer is waited for after the use before it was.
    uint64_t s_free[4];
    uint32_t qk_turn;                             // products whose S = Q K^T has been issued
    uint64_t o_full[2];
    uint64_t drain[2];
    uint64_t stage_done[2];                 // staged epilogue: the four warps of Q tile q have read their staging buffers out
    uint64_t work_full[2], work_empty[2];  // dynamic schedule: two-slot mailbox of claimed work indices
    long long work_k[2];
    uint32_t tmem_base;
    int abort_flag;
};

template <int kD, int kBlockN, int kQTiles>
struct Geometry {
    static constexpr int kChunks = kD / 64;                 // 64-element (128-byte) column blocks per row
    static constexpr int kQTileBytes = kBlockM * kD * 2;
    static constexpr int kKVTileBytes = kBlockN * kD * 2;
    static constexpr int kQChunkBytes = kBlockM * 128;
    static constexpr int kKVChunkBytes = kBlockN * 128;
    static constexpr int kColsS = kBlockN;                  // S columns a softmax thread owns: its whole row
    static constexpr int kColsO = kD;                       // O columns a softmax thread owns
    // Epilogue through shared memory: after the last V tile of a work item the ring holds one more slot that
    // nothing is loaded into; the softmax warps of Q tile q stage their 16-bit O rows in half q of it, kStageRows rows
    // of one 64-column block per warp at a time, and write them out with TMA stores (full 128-byte lines, rows
    // beyond N dropped by the copy engine).
    static constexpr int kStageBytesPerWarp = kKVTileBytes / 2 / 4;
    static constexpr int kStageRows = kStageBytesPerWarp / 128 < 32 ? kStageBytesPerWarp / 128 : 32;
    // P reaches the MMA warp in two parts: a thread announces its first kEarlyGroups groups of 16
    // probabilities (one K step of the P.V product each) while it still computes the rest.
    static constexpr int kGroups = kColsS / 16;
    // With eight groups five go first: the three that follow are the three K steps of P.V that remain on the chain behind
    // the softmax (measured 1-1.5 % ahead of six and two; P.V of the early part has finished by the time the rest arrives).
    static constexpr int kEarlyGroups = kGroups >= 8 ? (kGroups * 5) / 8 : kGroups >= 4 ? (kGroups * 3) / 4 : kGroups / 2;
    static constexpr int kSoftmaxWarps = kQTiles * 4;
    static constexpr int kTileThreads = 128;                // softmax threads of one Q tile
    static constexpr int kThreads = kSoftmaxWarps * 32 + 128;  // plus one warpgroup: producer, MMA warps, idle warp(s)
    // Registers: the launch gives every thread 65536 / kThreads rounded down to a multiple of 8.  With two Q tiles
    // that is 168 (384 threads): the last warpgroup hands registers back and the softmax warpgroups take them
    // (256 * 200 + 128 * 104 = 384 * 168).
    static constexpr bool kRebalance = (kQTiles == 2);
    static constexpr int kRegsOther = 104;
    static constexpr int kRegsSoftmax = 200;
    static constexpr int kTmemCols = 512;
    // Tensor memory: O_q (fp32, kD columns) at kTmemO + kD q, at the top; below it kSBufs buffers of kBlockN columns
    // for S (fp32), buffer b at kTmemS + kBlockN b; the P of a product overwrites the first half of its S buffer.
    static constexpr int kTmemO = kTmemCols - kQTiles * kD;
    static constexpr int kTmemS = 0;
    static constexpr int kSBufs = kTmemO / kBlockN < 4 ? kTmemO / kBlockN : 4;
    // As many buffers as tiles: buffer q belongs to tile q, and S_q of the next step can only follow P_q V of this
    // one.  More buffers than tiles: product n (counted over both tiles, in the order (step, tile)) uses buffer
    // n mod kSBufs, and a tile's next S product is issued before the MMA lane waits for the tile's present P.
    static constexpr bool kEarlyQK = kSBufs > kQTiles;
    static_assert(kSBufs >= kQTiles, "one S buffer per Q tile at least");
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
        for (int b = 0; b < 4; ++b) ptx::mbar_init(&bar->s_free[b], 1);
        for (int q = 0; q < 2; ++q) {
            ptx::mbar_init(&bar->o_full[q], 1);
            for (int e = 0; e < 2; ++e) {
                ptx::mbar_init(&bar->s_full[q][e], 1);
                ptx::mbar_init(&bar->p_early[q][e], 4);   // one arrival per softmax warp of the tile
                ptx::mbar_init(&bar->p_full[q][e], 4);
                ptx::mbar_init(&bar->pv_done[q][e], 1);
            }
        }
        bar->qk_turn = 0;
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(&bar->work_full[i], 1);
            ptx::mbar_init(&bar->work_empty[i], kQTiles + G::kSoftmaxWarps);
        }
        ptx::mbar_init(&bar->stage_done[0], 4);
        ptx::mbar_init(&bar->stage_done[1], 4);
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

    // Which work item this CTA handles as its item number `it`.  Static schedule (Algorithm 2): the CTA walks the
    // units blockIdx.x, += gridDim.x; `slot` counts the positions of that walk (a unit holds one or two items).
    // Dynamic schedule: the producer warp claims the next unclaimed item from a global counter and passes it to the
    // other roles through a two-slot mailbox in shared memory, so a CTA that drew short items simply draws more of
    // them.  Algorithm 4's parity is the CTA's own count `it` on the static walk and the claim's round on the dynamic one.
    const bool dynamic = p.work_counter != nullptr;
    auto static_next = [&](int& slot, int it, WorkItem& w) -> bool {
        for (;;) {
            const Slot sl = static_slot(p.sched, (int)blockIdx.x, (int)gridDim.x, slot++);
            if (sl.kind == kSlotEnd) return false;
            if (sl.kind == kSlotItem) { w = make_item(p.sched, sl.bh, sl.q_item, it); return true; }
        }
    };
    auto claimed_item = [&](long long claim, int it) -> WorkItem {
        // The scan direction of a claimed item follows the round of its claim (claim index / grid size): the CTA's own
        // count while the CTAs stay in step, and independent of which CTA won the claim, so results are reproducible.
        (void)it;
        const Slot sl = claimed_slot(p.sched, claim);
        return make_item(p.sched, sl.bh, sl.q_item, (int)(claim / (long long)gridDim.x));
    };
    auto claim_work = [&](int it, bool& ok) -> long long {  // producer warp, all lanes (dynamic schedule)
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
    auto take_work = [&](int it, bool& ok, bool whole_warp) -> long long {  // MMA lanes (one thread), softmax warps (dynamic schedule)
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

    // Which S buffer a product uses, and how often that buffer was used before.  idx: products of all tiles before it,
    // in the order (item, step, tile); every role counts them the same way.
    struct Product { uint32_t idx; int buf; uint32_t use; };
    auto product_of = [&](int q, uint32_t idx) -> Product {
        if (G::kEarlyQK) return Product{idx, (int)(idx % (uint32_t)G::kSBufs), idx / (uint32_t)G::kSBufs};
        return Product{idx, q, 0u};
    };
    // Does Q tile qq of the item take part in step s (its K/V tile lies below the tile's diagonal, and the tile below N)?
    auto visits = [&](const WorkItem& w, int s, int qq) -> bool { return kv_tile_at(w, s) < (qq ? w.hi_q[1] : w.hi_q[0]); };

    if (warp >= G::kSoftmaxWarps) {
    // The last warpgroup (producer, MMA and idle warps) hands registers back in one instruction.  (Its three
    // roles below keep the indentation of the outer level.)
    if (G::kRebalance) ptx::reg_dealloc<G::kRegsOther>();
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
        int it = 0, slot = 0;
        for (; ok; ++it) {
            WorkItem w;
            if (dynamic) {
                const long long k = claim_work(it, ok);
                if (!ok || k < 0) break;
                w = claimed_item(k, it);
            } else if (!static_next(slot, it, w)) {
                break;
            }
            ok = ptx::warp_all(ptx::mbar_wait(&bar->q_empty, (it & 1) ^ 1, abort_flag, kSiteProducerQ));
            if (!ok) break;
            // Tensor coordinates of the item's head: (batch, head) for Q, (batch, head of its group) for K and V.
            const int b_idx = w.bh / p.sched.H, h_idx = w.bh % p.sched.H;
            const int h_kv = h_idx / (p.sched.H / p.kv_heads);
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
                        if (p.l2_policy) ptx::tma_load_4d_hint(dst, &tm_q, &bar->q_full, c * 64, w.row0 + q * kBlockM, h_idx, b_idx, pol_q);
                        else ptx::tma_load_4d(dst, &tm_q, &bar->q_full, c * 64, w.row0 + q * kBlockM, h_idx, b_idx);
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
                            if (p.l2_policy) ptx::tma_load_4d_hint(dst, tm, &bar->kv_full[ring.slot], c * 64, j * kBlockN, h_kv, b_idx, pol_kv);
                            else ptx::tma_load_4d(dst, tm, &bar->kv_full[ring.slot], c * 64, j * kBlockN, h_kv, b_idx);
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
        uint32_t n_all = 0, k_mine = 0;   // products so far: of all tiles, of this lane's tile
        bool ok = true;

        // Descriptors differ from a base only in the 16-byte-granular address field (the low bits).
        const uint64_t q_desc = ptx::smem_desc_sw128(q_base, 16, 1024) + (uint64_t)((q * G::kQTileBytes) >> 4);
        const uint64_t k_desc0 = ptx::smem_desc_sw128(kv_base, 16, 1024);
        const uint64_t v_desc0 = ptx::smem_desc_sw128(kv_base, G::kKVChunkBytes, 1024);
        const uint32_t o_tmem = tmem + G::kTmemO + kD * q;
        auto issue_qk = [&](int slot, int buf) {
            const uint32_t s_tmem = tmem + G::kTmemS + kBlockN * buf;
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
        auto issue_pv = [&](int slot, int buf, uint32_t accumulate, int late) {
            const uint32_t s_tmem = tmem + G::kTmemS + kBlockN * buf;
            const uint64_t b0 = v_desc0 + (uint64_t)((slot * G::kKVTileBytes) >> 4);
#pragma unroll
            for (int kk = 0; kk < kBlockN / 16; ++kk) {
                if (((kk % G::kGroups) >= G::kEarlyGroups) != (late != 0)) continue;
                ptx::mma_ts(o_tmem, s_tmem + kk * 8, b0 + (uint64_t)(kk * ((16 * 128) >> 4)), idesc_pv,
                            accumulate | (late != 0) | (kk != 0));
            }
        };

        // More S buffers than tiles: before S of a product goes into a buffer, the products before it have had their S
        // issued (the lanes take turns), and the P.V product that used the buffer last has completed.
        auto buffer_free = [&](const Product& pr) -> bool {
            if (!ptx::spin_until_equal(&bar->qk_turn, pr.idx, abort_flag, kSiteMmaTurn)) return false;
            return pr.use == 0 || ptx::mbar_wait(&bar->s_free[pr.buf], (pr.use - 1) & 1u, abort_flag, kSiteMmaSFree);
        };

        // The elected lane runs the whole loop: every wait, issue and commit below is a single
        // thread's, with no warp votes or re-convergence between the MMA batches.
        if (ptx::elect_one()) {
            const long long clk_begin = clock64();
            SAW_PROF_DECL;
            int it = 0, slot = 0;
            for (; ok; ++it) {
                WorkItem w;
                if (dynamic) {
                    const long long k = take_work(it, ok, false);
                    if (!ok || k < 0) break;
                    w = claimed_item(k, it);
                } else if (!static_next(slot, it, w)) {
                    break;
                }
                const int hi_mine = q ? w.hi_q[1] : w.hi_q[0];
                SAW_PROF(0);
                if (!ptx::mbar_wait(&bar->q_full, it & 1, abort_flag, kSiteMmaQ)) { ok = false; break; }
                SAW_PROF(1);
                // K tile of step 0
                const int slot_k = ring.slot;
                if (!ptx::mbar_wait(&bar->kv_full[slot_k], ring.phase, abort_flag, kSiteMmaKV)) { ok = false; break; }
                ring.advance(stages);
                if (visits(w, 0, q)) {
                    const Product first = product_of(q, n_all + ((q == 1 && visits(w, 0, 0)) ? 1u : 0u));
                    if (G::kEarlyQK && !buffer_free(first)) { ok = false; break; }
                    ptx::tc_fence_after();
                    issue_qk(slot_k, first.buf);
                    ptx::mma_commit(&bar->s_full[q][k_mine & 1u]);
                    if (G::kEarlyQK) ptx::st_release_cta(&bar->qk_turn, first.idx + 1);
                }
                ptx::mma_commit(&bar->kv_empty[slot_k]);
                if (w.hi == 1) ptx::mma_commit(&bar->q_empty);
                uint32_t pv_started = 0;
                for (int s = 0; ok && s < w.hi; ++s) {
                    const bool has_next = s + 1 < w.hi;
                    const bool mine = visits(w, s, q);
                    const bool mine_next = has_next && visits(w, s + 1, q);
                    const uint32_t in_step = (uint32_t)visits(w, s, 0) + (kQTiles == 2 ? (uint32_t)visits(w, s, 1) : 0u);
                    const Product cur = product_of(q, n_all + ((q == 1 && visits(w, s, 0)) ? 1u : 0u));
                    const Product nxt = product_of(q, n_all + in_step + ((q == 1 && has_next && visits(w, s + 1, 0)) ? 1u : 0u));
                    const uint32_t k_next = k_mine + (mine ? 1u : 0u);   // the tile's product count at its next product
                    const uint32_t e_cur = k_mine & 1u, ph_cur = (k_mine >> 1) & 1u;
                    const int slot_v = ring.slot;
                    const uint32_t phase_v = ring.phase;
                    ring.advance(stages);
                    int slot_kn = 0;
                    uint32_t phase_kn = 0;
                    if (has_next) { slot_kn = ring.slot; phase_kn = ring.phase; ring.advance(stages); }
                    SAW_PROF(0);
                    if (G::kEarlyQK) {
                        // S of the tile's next step first, into a buffer whose last P has been read; then P.V of this step.
                        if (has_next) {
                            if (!ptx::mbar_wait(&bar->kv_full[slot_kn], phase_kn, abort_flag, kSiteMmaKV)) { ok = false; break; }
                            if (mine_next) {
                                if (!buffer_free(nxt)) { ok = false; break; }
                                ptx::tc_fence_after();
                                issue_qk(slot_kn, nxt.buf);
                                ptx::mma_commit(&bar->s_full[q][k_next & 1u]);
                                ptx::st_release_cta(&bar->qk_turn, nxt.idx + 1);
                                SAW_PROF(7);
                            }
                            ptx::mma_commit(&bar->kv_empty[slot_kn]);
                            if (s + 2 == w.hi) ptx::mma_commit(&bar->q_empty);  // the item's last S product is issued
                        }
                        if (!ptx::mbar_wait(&bar->kv_full[slot_v], phase_v, abort_flag, kSiteMmaKV)) { ok = false; break; }
                        SAW_PROF(2);
                        if (mine) {
                            if (!ptx::mbar_wait(&bar->p_early[q][e_cur], ph_cur, abort_flag, kSiteMmaP)) { ok = false; break; }
                            SAW_PROF(3);
                            ptx::tc_fence_after();
                            issue_pv(slot_v, cur.buf, pv_started, 0);
                            SAW_PROF(4);
                            if (!ptx::mbar_wait(&bar->p_full[q][e_cur], ph_cur, abort_flag, kSiteMmaP)) { ok = false; break; }
                            SAW_PROF(5);
                            ptx::tc_fence_after();
                            issue_pv(slot_v, cur.buf, pv_started, 1);
                            pv_started = 1;
                            ptx::mma_commit(&bar->s_free[cur.buf]);
                            ptx::mma_commit(&bar->pv_done[q][e_cur]);
                            SAW_PROF(6);
                        }
                        ptx::mma_commit(&bar->kv_empty[slot_v]);
                    } else {
                        if (!ptx::mbar_wait(&bar->kv_full[slot_v], phase_v, abort_flag, kSiteMmaKV)) { ok = false; break; }
                        if (has_next && !ptx::mbar_wait(&bar->kv_full[slot_kn], phase_kn, abort_flag, kSiteMmaKV)) { ok = false; break; }
                        SAW_PROF(2);
                        if (mine) {
                            if (!ptx::mbar_wait(&bar->p_early[q][e_cur], ph_cur, abort_flag, kSiteMmaP)) { ok = false; break; }
                            SAW_PROF(3);
                            ptx::tc_fence_after();
                            issue_pv(slot_v, cur.buf, pv_started, 0);
                            SAW_PROF(4);
                            if (!ptx::mbar_wait(&bar->p_full[q][e_cur], ph_cur, abort_flag, kSiteMmaP)) { ok = false; break; }
                            SAW_PROF(5);
                            ptx::tc_fence_after();
                            issue_pv(slot_v, cur.buf, pv_started, 1);
                            pv_started = 1;
                            SAW_PROF(6);
                        }
                        if (mine_next) {
                            ptx::tc_fence_after();
                            issue_qk(slot_kn, nxt.buf);
                            ptx::mma_commit(&bar->s_full[q][k_next & 1u]);
                            SAW_PROF(7);
                        }
                        // Every lane commits every slot, used by its tile or not: the slot's count is the number of lanes.
                        ptx::mma_commit(&bar->kv_empty[slot_v]);
                        if (has_next) {
                            ptx::mma_commit(&bar->kv_empty[slot_kn]);
                            if (s + 2 == w.hi) ptx::mma_commit(&bar->q_empty);  // the item's last S product is issued
                        }
                    }
                    n_all += in_step;
                    k_mine += mine ? 1u : 0u;
                    SAW_PROF(8);
                }
                if (!ok) break;
                if (hi_mine > 0) ptx::mma_commit(&bar->o_full[q]);
                // The item's staging slot is not this lane's business: the softmax warps take it over from the producer
                // and hand it back.  (A lane whose tile lies beyond N has nothing to wait for in an item and may be a whole
                // item ahead of the softmax warps, so it must not count towards that slot's release.)
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
        if (G::kRebalance) ptx::reg_alloc<G::kRegsSoftmax>();
        constexpr int kColsS = G::kColsS, kColsO = G::kColsO;
        // (Measured per tile shape: with 64-row K/V tiles at d = 64 three pairs in eight, with a single Q tile at d = 128,
        // where the softmax sets the step as well, one in eight.)
        constexpr int kExpPolyMask = kD == 64 ? (kBlockN == 64 ? 0x49 : SAW_EXP_POLY_MASK_D64)
                                              : (kQTiles == 1 ? 0x01 : SAW_EXP_POLY_MASK_D128);
        const int q = warp >> 2;                       // which Q tile this thread works on
        const int r_in_tile = (warp & 3) * 32 + lane;  // row inside the tile = TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_o = tmem + lane_base + G::kTmemO + kD * q;
        const float scale_log2 = p.scale_log2;
        const int N = p.sched.N;
        uint32_t o_phase = 0;
        uint32_t n_all = 0, k_mine = 0;   // products so far: of all tiles, of this thread's tile
        bool ok = true;
        int it = 0, slot = 0;
        Ring ring;                 // position of the next work item's first K tile in the K/V ring
        uint32_t stage_phase = 0;
        SAW_PROF_DECL;
        for (; ok; ++it) {
            WorkItem w;
            if (dynamic) {
                const long long k = take_work(it, ok, true);
                if (!ok || k < 0) break;
                w = claimed_item(k, it);
            } else if (!static_next(slot, it, w)) {
                break;
            }
            const int hi_mine = q ? w.hi_q[1] : w.hi_q[0];
            ring.advance_by(2 * w.hi, stages);   // now at the item's staging slot
            const Ring stage = ring;
            ring.advance(stages);
            if (hi_mine == 0) {   // the tile lies beyond N: only the other tile's products count
                n_all += (uint32_t)(w.hi_q[0] + w.hi_q[1]);
                continue;
            }
            const int tile_row0 = w.row0 + q * kBlockM;
            const int row = tile_row0 + r_in_tile;
            float m_ref = -INFINITY;   // the max the exponents are taken against (log2 units)
            float l = 0.f;             // running sum of this thread's probabilities
            bool first = true;
            for (int s = 0; s < w.hi; ++s) {
                const int j = kv_tile_at(w, s);
                const uint32_t in_step = (uint32_t)visits(w, s, 0) + (kQTiles == 2 ? (uint32_t)visits(w, s, 1) : 0u);
                if (j >= hi_mine) { n_all += in_step; continue; }
                const Product cur = product_of(q, n_all + ((q == 1 && visits(w, s, 0)) ? 1u : 0u));
                const uint32_t e_cur = k_mine & 1u, ph_cur = (k_mine >> 1) & 1u;
                n_all += in_step;
                const uint32_t t_s = tmem + lane_base + G::kTmemS + kBlockN * cur.buf;
                const uint32_t t_p = t_s;              // P overwrites the first half of the row's S columns
                SAW_PROF(0);
                const bool got_s = ptx::mbar_wait(&bar->s_full[q][e_cur], ph_cur, abort_flag, kSiteSoftmaxS);
                ptx::tc_fence_after();
                SAW_PROF(1);

                uint32_t sv[kColsS / 32][32];
#pragma unroll
                for (int c = 0; c < kColsS / 32; ++c) ptx::tmem_ld32(t_s + c * 32, sv[c]);
                ptx::tmem_wait_ld();
                SAW_PROF(2);

                if (p.negate) {   // a negative scale: work on -S with |scale|
#pragma unroll
                    for (int c = 0; c < kColsS / 32; ++c)
#pragma unroll
                        for (int i = 0; i < 32; ++i) sv[c][i] ^= 0x80000000u;
                }
                const int col0 = j * kBlockN;  // key index of the row's first column
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
                SAW_PROF(3);
                ok = ptx::warp_all(got_s);
                if (!ok) break;
                SAW_PROF(4);
                const float m_cand = fmaxf(m_ref, row_max * scale_log2);
                const bool need = (m_cand - m_ref) > kRescaleThreshold;
                if (__any_sync(0xffffffffu, need)) {
                    float alpha = 1.f;
                    if (need) {
                        alpha = ptx::ex2(m_ref - m_cand);  // 0 when nothing was accumulated yet
                        m_ref = m_cand;
                        l *= alpha;
                    }
                    if (!first) {
                        // O_q's last update must have completed.  It was issued before this S product, which is
                        // complete, unless S products run ahead: then the update has a barrier of its own.
                        if (G::kEarlyQK) {
                            ok = ptx::warp_all(ptx::mbar_wait(&bar->pv_done[q][(k_mine - 1) & 1u], ((k_mine - 1) >> 1) & 1u, abort_flag,
                                                              kSiteSoftmaxPvDone));
                            if (!ok) break;
                            ptx::tc_fence_after();
                        }
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
                }
                SAW_PROF(5);
                const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
                const ptx::f32x2 scale2 = ptx::pack_f32x2(scale_log2, scale_log2);
                const ptx::f32x2 neg_m2 = ptx::pack_f32x2(neg_m, neg_m);
                ptx::f32x2 l01 = ptx::pack_f32x2(0.f, 0.f), l23 = ptx::pack_f32x2(0.f, 0.f);
                // Groups of 16 probabilities (eight packed registers, one TMEM store each).  The store of a
                // group is issued after the exponentials of the next group, so that it never waits in the
                // instruction stream for MUFU results that are still in flight.
                uint32_t pk[G::kGroups][8];
                auto finish_group = [&](int g) {
                    ptx::tmem_st8(t_p + g * 8, pk[g]);
                    if (g == G::kEarlyGroups - 1) {
                        ptx::tmem_wait_st();
                        ptx::tc_fence_before();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(&bar->p_early[q][e_cur]);
                        SAW_PROF(6);
                    }
                };
#pragma unroll
                for (int g = 0; g < G::kGroups; ++g) {
                    const int c = g >> 1, h = g & 1;
#pragma unroll
                    for (int i = 0; i < 16; i += 4) {
                        // Four probabilities: x = S * scale * log2(e) - m as two packed FMAs, then 2^x on the MUFU
                        // or, for the pairs of the group that kExpPolyMask names, on the FMA pipe.
                        const ptx::f32x2 xa = ptx::fma2(ptx::pack_f32x2(__uint_as_float(sv[c][16 * h + i]), __uint_as_float(sv[c][16 * h + i + 1])), scale2, neg_m2);
                        const ptx::f32x2 xb = ptx::fma2(ptx::pack_f32x2(__uint_as_float(sv[c][16 * h + i + 2]), __uint_as_float(sv[c][16 * h + i + 3])), scale2, neg_m2);
                        float x0, x1, x2, x3, p0, p1, p2, p3;
                        ptx::unpack_f32x2(xa, x0, x1);
                        ptx::unpack_f32x2(xb, x2, x3);
                        if ((kExpPolyMask >> ((i >> 2) * 2)) & 1) ptx::exp2_poly_pair(x0, x1, p0, p1);
                        else { p0 = ptx::ex2(x0); p1 = ptx::ex2(x1); }
                        if ((kExpPolyMask >> ((i >> 2) * 2 + 1)) & 1) ptx::exp2_poly_pair(x2, x3, p2, p3);
                        else { p2 = ptx::ex2(x2); p3 = ptx::ex2(x3); }
                        l01 = ptx::add2(l01, ptx::pack_f32x2(p0, p1));
                        l23 = ptx::add2(l23, ptx::pack_f32x2(p2, p3));
                        pk[g][i / 2] = ptx::pack2<kBf16>(p0, p1);
                        pk[g][i / 2 + 1] = ptx::pack2<kBf16>(p2, p3);
                    }
                    if (g > 0) finish_group(g - 1);
                }
                finish_group(G::kGroups - 1);
                float l0, l1, l2, l3;
                ptx::unpack_f32x2(l01, l0, l1);
                ptx::unpack_f32x2(l23, l2, l3);
                l += (l0 + l1) + (l2 + l3);
                ptx::tmem_wait_st();
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&bar->p_full[q][e_cur]);
                SAW_PROF(7);
                first = false;
                ++k_mine;
            }
            if (!ok) break;
            // ---- epilogue: O_q / l -> 16 bit -> global
            SAW_PROF(0);
            const bool got_o = ptx::mbar_wait(&bar->o_full[q], o_phase, abort_flag, kSiteSoftmaxO);
            o_phase ^= 1u;
            ptx::tc_fence_after();
            SAW_PROF(9);
            ok = ptx::warp_all(got_o);
            if (!ok) break;
            const float inv_l = 1.f / l;
            // ln sum_j exp(scale * s_j) of the row: the probabilities were taken as 2^(x - m_ref), so the sum is 2^m_ref * l.
            if (p.lse != nullptr && row < N) p.lse[(size_t)w.bh * N + row] = (m_ref + log2f(l)) * 0.6931471805599453f;
            ok = ptx::warp_all(ptx::mbar_wait(&bar->kv_full[stage.slot], stage.phase, abort_flag, kSiteStageSlot));
            if (!ok) break;
            SAW_PROF(10);
            uint8_t* buf = kv_smem + (size_t)stage.slot * G::kKVTileBytes + (size_t)q * (G::kKVTileBytes / 2) +
                           (size_t)(warp & 3) * G::kStageBytesPerWarp;
            const int my_pass = lane / G::kStageRows, my_row = lane % G::kStageRows;
#pragma unroll
            for (int c64 = 0; c64 < kD / 64; ++c64) {
                uint32_t pk[32];   // this row's 64 columns of the block, 16-bit pairs
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    uint32_t ov[32];
                    ptx::tmem_ld32(t_o + c64 * 64 + hf * 32, ov);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; i += 2)
                        pk[hf * 16 + i / 2] = ptx::pack2<kBf16>(__uint_as_float(ov[i]) * inv_l, __uint_as_float(ov[i + 1]) * inv_l);
                }
#pragma unroll 1
                for (int ps = 0; ps < 32 / G::kStageRows; ++ps) {
                    if (my_pass == ps) {
                        // 128-byte rows, eight to a 1024-byte swizzle atom: 16-byte piece i of row r sits at piece i ^ (r & 7)
                        uint4* dst_row = reinterpret_cast<uint4*>(buf + my_row * 128);
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            dst_row[i ^ (my_row & 7)] = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
                    }
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    const int y0 = tile_row0 + (warp & 3) * 32 + ps * G::kStageRows;
                    if (y0 < N && ptx::elect_one()) {   // rows of the box beyond N are dropped by the copy
                        ptx::tma_store_4d(&tm_o, buf, c64 * 64, y0, w.bh % p.sched.H, w.bh / p.sched.H);
                        ptx::bulk_commit_group();
                        ptx::bulk_wait_group_read0();   // the buffer may be written again
                    }
                    __syncwarp();
                }
            }
            SAW_PROF(11);
            // The slot goes back to the producer once the four warps of the tile have read their buffers out.
            if (lane == 0) ptx::mbar_arrive(&bar->stage_done[q]);
            if ((warp & 3) == 0) {
                ok = ptx::warp_all(ptx::mbar_wait(&bar->stage_done[q], stage_phase, abort_flag, kSiteStageDone));
                // One arrival per Q tile of the item; a second tile that lies beyond N has no warps at work: the first
                // tile's warp arrives for it, after its own rows have left the slot.
                if (ok && lane == 0) {
                    ptx::mbar_arrive(&bar->kv_empty[stage.slot]);
                    if (kQTiles == 2 && q == 0 && w.hi_q[1] == 0) ptx::mbar_arrive(&bar->kv_empty[stage.slot]);
                }
            }
            stage_phase ^= 1u;
            if (!ok) break;
            ptx::tc_fence_before();  // ordered before this thread's next arrive on p_full, which lets O_q be overwritten
            SAW_PROF(8);
        }
        ptx::bulk_wait_group0();   // this thread's TMA stores have landed before the CTA ends
        SAW_PROF_WRITE(12, q == 0 && r_in_tile == 0);
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
