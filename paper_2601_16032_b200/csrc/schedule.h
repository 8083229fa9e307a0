// Tile schedule of the attention forward pass, shared by the host (plan, trace) and the kernel.
//
// Work is cut into items of W = q_tiles * 128 query rows of one (batch, head).  A persistent grid of
// G = min(n_units, SM count) CTAs walks the linear unit index u = blockIdx.x, += G (Algorithm 2 of
// the paper).  A unit is one item or, with pairing, two items of one head that the CTA handles one
// after the other:
//   mirrored pairs  (q, n_q-1-q): the Q block that lies n_q-1-p blocks into the head, then the one
//                   that lies p blocks into it.  Under the causal mask the two scan n_q+1 blocks'
//                   worth of K/V tiles between them whatever p is, so every unit takes the same
//                   time and the static walk stays balanced and in step;
//   adjacent pairs  (2p, 2p+1): two neighbouring Q blocks per trip of the CTA's loop.
// The CTA counts the items it has handled (`it`, Algorithm 4's i_local): item number `it` scans its
// K/V tiles first-to-last, or, in the sawtooth order and for odd `it`, last-to-first.  With pairs
// that is first-to-last for a unit's first item and last-to-first for its second.  Under the causal
// mask only K/V tiles that hold a key visible to some row of the item are visited.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define SAW_HD __host__ __device__ __forceinline__
#else
#define SAW_HD inline
#endif

namespace sawtooth {

constexpr int kBlockM = 128;  // query rows per MMA tile (one TMEM lane per row)

enum Pairing { kPairNone = 0, kPairMirrored = 1, kPairAdjacent = 2 };

struct SchedParams {
    int B, H, N;
    int q_tiles;      // 128-row Q tiles per work item (1 or 2)
    int block_n;      // K/V rows per tile
    int causal;       // 0 / 1
    int sawtooth;     // 0 = cyclic, 1 = sawtooth
    int head_fastest; // 0: u = (b*H + h)*units_per_head + p    1: u = (b*units_per_head + p)*H + h
    int heavy_first;  // 1: digit p counts the Q blocks of a head from the last (most K/V tiles under the causal mask) to the first
    int pairing;      // Pairing
    int n_q;          // work items per head = ceil(N / W)
    int units_per_head; // n_q, or ceil(n_q / 2) with pairing
    long long n_work;   // B * H * n_q
    long long n_units;  // B * H * units_per_head
};

struct WorkItem {
    int bh;        // b*H + h
    int q_item;    // index of the work item inside its head
    int row0;      // first query row of the item
    int backward;  // scan direction of this CTA iteration
    int hi;        // K/V tiles 0..hi-1 are visited by the item
    int hi_q[2];   // per 128-row Q tile: tiles 0..hi_q-1 are needed (0: tile lies beyond N)
};

// Where slot s of a CTA's walk lands.
enum SlotKind { kSlotItem = 0, kSlotEmpty = 1, kSlotEnd = 2 };
struct Slot {
    int kind;      // SlotKind: an item, nothing (the second half of a unit that holds one item), or the end of the walk
    int bh;
    int q_item;
};

SAW_HD int ceil_div_i(int a, int b) { return (a + b - 1) / b; }

SAW_HD SchedParams make_sched(int B, int H, int N, int q_tiles, int block_n, int causal, int sawtooth, int head_fastest,
                              int heavy_first = 0, int pairing = kPairNone) {
    SchedParams p;
    p.heavy_first = heavy_first;
    p.pairing = pairing;
    p.B = B; p.H = H; p.N = N; p.q_tiles = q_tiles; p.block_n = block_n;
    p.causal = causal; p.sawtooth = sawtooth; p.head_fastest = head_fastest;
    p.n_q = ceil_div_i(N, q_tiles * kBlockM);
    p.units_per_head = pairing == kPairNone ? p.n_q : ceil_div_i(p.n_q, 2);
    p.n_work = (long long)B * H * p.n_q;
    p.n_units = (long long)B * H * p.units_per_head;
    return p;
}

// Linear unit index -> (b*H + h, position of the unit inside its head).
SAW_HD void split_unit(const SchedParams& p, long long u, int& bh, int& pos) {
    if (!p.head_fastest) {
        pos = (int)(u % p.units_per_head);
        bh = (int)(u / p.units_per_head);
    } else {
        const int h = (int)(u % p.H);
        const long long r = u / p.H;
        pos = (int)(r % p.units_per_head);
        bh = (int)(r / p.units_per_head) * p.H + h;
    }
}

// Slot s (0, 1, 2, ...) of the static walk of CTA `cta` in a grid of G (Algorithm 2).
SAW_HD Slot static_slot(const SchedParams& p, int cta, int G, int s) {
    Slot r;
    const int members = p.pairing == kPairNone ? 1 : 2;
    const long long u = (long long)cta + (long long)(s / members) * G;
    if (u >= p.n_units) { r.kind = kSlotEnd; r.bh = 0; r.q_item = 0; return r; }
    int pos;
    split_unit(p, u, r.bh, pos);
    const int m = s % members;
    r.kind = kSlotItem;
    if (p.pairing == kPairNone) {
        r.q_item = p.heavy_first ? p.n_q - 1 - pos : pos;
    } else if (p.pairing == kPairMirrored) {
        r.q_item = m == 0 ? p.n_q - 1 - pos : pos;
        if (m == 1 && p.n_q - 1 - pos == pos) r.kind = kSlotEmpty;   // the middle block of an odd count stands alone
    } else {
        r.q_item = 2 * pos + m;
        if (r.q_item >= p.n_q) r.kind = kSlotEmpty;
    }
    return r;
}

// Item `claim` (0, 1, 2, ...) of the dynamic schedule, where CTAs claim single items in index order.
SAW_HD Slot claimed_slot(const SchedParams& p, long long claim) {
    Slot r;
    if (claim >= p.n_work) { r.kind = kSlotEnd; r.bh = 0; r.q_item = 0; return r; }
    int pos;
    split_unit(p, claim, r.bh, pos);   // no pairing here: units are items
    r.kind = kSlotItem;
    r.q_item = p.heavy_first ? p.n_q - 1 - pos : pos;
    return r;
}

// The item at (bh, q_item), handled as item number `it` of its CTA.
SAW_HD WorkItem make_item(const SchedParams& p, int bh, int q_item, int it) {
    WorkItem w;
    w.bh = bh;
    w.q_item = q_item;
    w.row0 = q_item * p.q_tiles * kBlockM;
    w.backward = (p.sawtooth && (it & 1)) ? 1 : 0;
    const int n_kv = ceil_div_i(p.N, p.block_n);
    w.hi = 0;
#if defined(__CUDA_ARCH__)
#pragma unroll
#endif
    for (int q = 0; q < 2; ++q) {
        int h = 0;
        const int r = w.row0 + q * kBlockM;
        if (q < p.q_tiles && r < p.N) {
            if (p.causal) {
                const int last_excl = (r + kBlockM < p.N) ? r + kBlockM : p.N;
                h = ceil_div_i(last_excl, p.block_n);
            } else {
                h = n_kv;
            }
        }
        w.hi_q[q] = h;
        if (h > w.hi) w.hi = h;
    }
    return w;
}

// K/V tile visited at step s (0 <= s < hi) of the item's scan.
SAW_HD int kv_tile_at(const WorkItem& w, int s) { return w.backward ? (w.hi - 1 - s) : s; }

}  // namespace sawtooth
