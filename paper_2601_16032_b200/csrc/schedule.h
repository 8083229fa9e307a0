// Tile schedule of the attention forward pass, shared by the host (plan, trace) and the kernel.
//
// Work is cut into items of W = q_tiles * 128 query rows of one (batch, head).  A persistent grid of
// G = min(n_work, SM count) CTAs walks the linear item index k = blockIdx.x, += G (Algorithm 2 of
// the paper).  Iteration number `it` of a CTA scans its K/V tiles first-to-last, or, in the sawtooth
// order and for odd `it`, last-to-first (Algorithm 4).  Under the causal mask only K/V tiles that
// hold a key visible to some row of the item are visited.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define SAW_HD __host__ __device__ __forceinline__
#else
#define SAW_HD inline
#endif

namespace sawtooth {

constexpr int kBlockM = 128;  // query rows per MMA tile (one TMEM lane per row)

struct SchedParams {
    int B, H, N;
    int q_tiles;      // 128-row Q tiles per work item (1 or 2)
    int block_n;      // K/V rows per tile
    int causal;       // 0 / 1
    int sawtooth;     // 0 = cyclic, 1 = sawtooth
    int head_fastest; // 0: k = (b*H + h)*n_q + t    1: k = (b*n_q + t)*H + h
    int heavy_first;  // 1: digit t counts the Q blocks of a head from the last (most K/V tiles under the causal mask) to the first
    int n_q;          // work items per head = ceil(N / W)
    long long n_work; // B * H * n_q
};

struct WorkItem {
    int bh;        // b*H + h
    int q_item;    // index of the work item inside its head
    int row0;      // first query row of the item
    int backward;  // scan direction of this CTA iteration
    int hi;        // K/V tiles 0..hi-1 are visited by the item
    int hi_q[2];   // per 128-row Q tile: tiles 0..hi_q-1 are needed (0: tile lies beyond N)
};

SAW_HD int ceil_div_i(int a, int b) { return (a + b - 1) / b; }

SAW_HD SchedParams make_sched(int B, int H, int N, int q_tiles, int block_n, int causal, int sawtooth, int head_fastest,
                              int heavy_first = 0) {
    SchedParams p;
    p.heavy_first = heavy_first;
    p.B = B; p.H = H; p.N = N; p.q_tiles = q_tiles; p.block_n = block_n;
    p.causal = causal; p.sawtooth = sawtooth; p.head_fastest = head_fastest;
    p.n_q = ceil_div_i(N, q_tiles * kBlockM);
    p.n_work = (long long)B * H * p.n_q;
    return p;
}

// Item k handled as iteration `it` of its CTA.
SAW_HD WorkItem decode_work(const SchedParams& p, long long k, int it) {
    WorkItem w;
    if (!p.head_fastest) {
        w.q_item = (int)(k % p.n_q);
        w.bh = (int)(k / p.n_q);
    } else {
        const int h = (int)(k % p.H);
        const long long r = k / p.H;
        w.q_item = (int)(r % p.n_q);
        w.bh = (int)(r / p.n_q) * p.H + h;
    }
    if (p.heavy_first) w.q_item = p.n_q - 1 - w.q_item;
    w.row0 = w.q_item * p.q_tiles * kBlockM;
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
