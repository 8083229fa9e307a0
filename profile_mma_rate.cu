// Measuring aid: SM cycles per tcgen05.mma (kind::f16, bf16 operands, fp32 accumulate, M = 128, K = 16) as the attention
// kernel issues them, for N = 128 and 64, with both operands in shared memory (the form of S = Q K^T) and with A in
// tensor memory (the form of O += P V), issued by one to four threads of a CTA at once, one CTA per SM.
//
//     nvcc -std=c++17 -O3 -gencode arch=compute_100a,code=sm_100a -o profile_mma_rate profile_mma_rate.cu && ./profile_mma_rate
//
// Operands are zero-filled shared memory laid out like the kernel's tiles (128-byte swizzle, K-major); the products are
// discarded.  Every wait is bounded; a wait that runs out shows as "status 1".
#include <cstdio>
#include <cstdlib>

#include "paper_2601_16032_b200/csrc/ptx.cuh"
using namespace sawtooth;

constexpr int kThreads = 160;          // warp 0 owns the TMEM allocation, warps 1..4 issue
constexpr int kSmemBytes = 96 * 1024;  // A: 2 chunks of 128 rows x 128 bytes; B: up to 256 rows

// a_in_tmem: 0 = every MMA takes A from shared memory, 1 = from tensor memory, 2 = a thread alternates the two forms,
// 3 = even issuing threads use shared memory, odd ones tensor memory.
__global__ void __launch_bounds__(kThreads, 1) mma_rate(int n_cols, int a_in_tmem, int batches, int issuers, unsigned long long* out, int* status) {
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ uint64_t done[4];
    __shared__ uint32_t tmem_base;
    __shared__ int abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5;
    for (int i = tid; i < kSmemBytes / 16; i += kThreads) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        for (int i = 0; i < 4; ++i) ptx::mbar_init(&done[i], 1);
        abort_flag = 0;
        ptx::fence_mbar_init();
    }
    ptx::fence_proxy_async_smem();
    if (warp == 0) { ptx::tmem_alloc(&tmem_base, 512); ptx::tmem_relinquish(); }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = tmem_base;
    if (warp >= 1 && warp <= issuers && ptx::elect_one()) {
        const int me = warp - 1;
        const uint32_t base = ptx::smem_u32(smem);
        const uint64_t a_desc = ptx::smem_desc_sw128(base, 16, 1024);
        const uint64_t b_desc = ptx::smem_desc_sw128(base + 32768, 16, 1024);
        const uint32_t idesc = ptx::instr_desc_f16(1, 0, 128, (uint32_t)n_cols);
        const long long t0 = clock64();
        for (int it = 0; it < batches; ++it) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {   // eight K steps accumulating into this thread's own 128 columns
                const int c = i >> 2, kk = i & 3;
                const uint64_t ad = a_desc + (uint64_t)((c * 16384 + kk * 32) >> 4);
                const uint64_t bd = b_desc + (uint64_t)((c * 16384 + kk * 32) >> 4);
                const bool from_tmem = a_in_tmem == 1 || (a_in_tmem == 2 && (i & 1)) || (a_in_tmem == 3 && (me & 1));
                // The two forms of a mix accumulate into columns of their own: 256 columns per thread then (at most two threads).
                const uint32_t d = a_in_tmem == 2 ? tmem + me * 256 + (i & 1) * 128 : tmem + me * 128;
                if (from_tmem) ptx::mma_ts(d, tmem + ((me + 1) & 3) * 128 + i * 8, bd, idesc, 1);
                else ptx::mma_ss(d, ad, bd, idesc, 1);
            }
        }
        ptx::mma_commit(&done[me]);
        const bool ok = ptx::mbar_wait(&done[me], 0, &abort_flag, 1);
        const long long t1 = clock64();
        if (blockIdx.x == 0 && me == 0) out[0] = (unsigned long long)(t1 - t0);
        if (!ok) atomicExch(status, 1);
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) { ptx::tc_fence_after(); ptx::tmem_dealloc(tmem, 512); }
}

// The same measurement with the shared-memory operands in the other K-major layouts the descriptor knows: rows of 64
// bytes (64-byte swizzle), rows of 32 bytes (32-byte swizzle: one row is exactly one K step) and unswizzled 8 x 16-byte
// core matrices.  layout: 0 = 128-byte swizzle, 1 = 64-byte, 2 = 32-byte, 3 = none.  One issuing thread, N = 128.
__device__ __forceinline__ uint64_t desc_for_step(uint32_t base, int layout, int i) {
    // address of K step i (16 elements, 32 bytes of every row) of a 128-row operand, and the strides of its layout
    uint32_t addr, lbo, sbo;
    uint64_t swizzle;
    if (layout == 0) { addr = base + (i >> 2) * 16384 + (i & 3) * 32; lbo = 16; sbo = 1024; swizzle = 2; }
    else if (layout == 1) { addr = base + (i >> 1) * 8192 + (i & 1) * 32; lbo = 16; sbo = 512; swizzle = 4; }
    else if (layout == 2) { addr = base + i * 4096; lbo = 16; sbo = 256; swizzle = 6; }
    else { addr = base + i * 4096; lbo = 128; sbo = 256; swizzle = 0; }
    uint64_t d = 0;
    d |= static_cast<uint64_t>((addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((lbo >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>((sbo >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;
    d |= swizzle << 61;
    return d;
}
__global__ void __launch_bounds__(kThreads, 1) mma_rate_layout(int a_layout, int b_layout, int a_in_tmem, int batches, unsigned long long* out, int* status) {
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ uint64_t done;
    __shared__ uint32_t tmem_base;
    __shared__ int abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5;
    for (int i = tid; i < kSmemBytes / 16; i += kThreads) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) { ptx::mbar_init(&done, 1); abort_flag = 0; ptx::fence_mbar_init(); }
    ptx::fence_proxy_async_smem();
    if (warp == 0) { ptx::tmem_alloc(&tmem_base, 512); ptx::tmem_relinquish(); }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = tmem_base;
    if (warp == 1 && ptx::elect_one()) {
        const uint32_t base = ptx::smem_u32(smem);
        uint64_t ad[8], bd[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) { ad[i] = desc_for_step(base, a_layout, i); bd[i] = desc_for_step(base + 32768, b_layout, i); }
        const uint32_t idesc = ptx::instr_desc_f16(1, 0, 128, 128);
        const long long t0 = clock64();
        for (int it = 0; it < batches; ++it) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (a_in_tmem) ptx::mma_ts(tmem, tmem + 128 + i * 8, bd[i], idesc, 1);
                else ptx::mma_ss(tmem, ad[i], bd[i], idesc, 1);
            }
        }
        ptx::mma_commit(&done);
        const bool ok = ptx::mbar_wait(&done, 0, &abort_flag, 1);
        const long long t1 = clock64();
        if (blockIdx.x == 0) out[0] = (unsigned long long)(t1 - t0);
        if (!ok) atomicExch(status, 1);
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) { ptx::tc_fence_after(); ptx::tmem_dealloc(tmem, 512); }
}

// The same measurement for the two-SM form (cta_group::2): a cluster of two CTAs, M = 256 (128 rows in each CTA's tensor
// memory), N = 128 with each CTA holding 64 of the 128 B rows in its own shared memory; one thread of the cluster's first
// CTA issues for both.
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
mma_rate_pair(int a_in_tmem, int batches, unsigned long long* out, int* status) {
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ uint64_t done;
    __shared__ uint32_t tmem_base;
    __shared__ int abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5;
    for (int i = tid; i < kSmemBytes / 16; i += kThreads) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) { ptx::mbar_init(&done, 1); abort_flag = 0; ptx::fence_mbar_init(); }
    ptx::fence_proxy_async_smem();
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(ptx::smem_u32(&tmem_base)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    ptx::tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    ptx::tc_fence_after();
    const uint32_t tmem = tmem_base;
    if (cluster_rank() == 0 && warp == 1 && ptx::elect_one()) {
        const uint32_t base = ptx::smem_u32(smem);
        const uint64_t a_desc = ptx::smem_desc_sw128(base, 16, 1024);
        const uint64_t b_desc = ptx::smem_desc_sw128(base + 32768, 16, 1024);
        const uint32_t idesc = ptx::instr_desc_f16(1, 0, 256, 128);
        const long long t0 = clock64();
        for (int it = 0; it < batches; ++it) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int c = i >> 2, kk = i & 3;
                const uint64_t ad = a_desc + (uint64_t)((c * 16384 + kk * 32) >> 4);
                const uint64_t bd = b_desc + (uint64_t)((c * 8192 + kk * 32) >> 4);
                if (a_in_tmem)
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                                 "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                                 ::"r"(tmem), "r"(tmem + 256 + i * 8), "l"(bd), "r"(idesc), "r"(1u) : "memory");
                else
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                                 "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                 ::"r"(tmem), "l"(ad), "l"(bd), "r"(idesc), "r"(1u) : "memory");
            }
        }
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(ptx::smem_u32(&done)) : "memory");
        const bool ok = ptx::mbar_wait(&done, 0, &abort_flag, 1);
        const long long t1 = clock64();
        if (blockIdx.x == 0) out[0] = (unsigned long long)(t1 - t0);
        if (!ok) atomicExch(status, 1);
    }
    ptx::tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 0) {
        ptx::tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    }
}

int main() {
    unsigned long long* out;
    int* status;
    if (cudaMalloc(&out, 8) != cudaSuccess || cudaMalloc(&status, 4) != cudaSuccess) { printf("no CUDA device\n"); return 1; }
    cudaMemset(status, 0, 4);
    cudaFuncSetAttribute(mma_rate, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    int sms = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0);
    const int batches = 2000;
    printf("cycles per 128 x N x 16 MMA (all issuing threads together), %d CTAs\n", sms);
    for (int a_in_tmem = 0; a_in_tmem < 4; ++a_in_tmem)
        for (int n : {128, 64})
            for (int issuers = 1; issuers <= 4; ++issuers) {
                if (a_in_tmem == 2 && issuers > 2) continue;   // 256 columns per thread
                for (int rep = 0; rep < 2; ++rep) {
                    mma_rate<<<sms, kThreads, kSmemBytes>>>(n, a_in_tmem, batches, issuers, out, status);
                    cudaError_t e = cudaDeviceSynchronize();
                    if (e != cudaSuccess) { printf("error %s\n", cudaGetErrorString(e)); return 1; }
                }
                unsigned long long cycles = 0;
                int st = 0;
                cudaMemcpy(&cycles, out, 8, cudaMemcpyDeviceToHost);
                cudaMemcpy(&st, status, 4, cudaMemcpyDeviceToHost);
                const double per = (double)cycles / (8.0 * batches * issuers);
                const char* where[4] = {"smem", "TMEM", "smem and TMEM alternating in each thread", "smem (even threads) / TMEM (odd threads)"};
                printf("A in %s, N = %3d, %d issuing thread(s): %6.1f cycles per MMA, %5.0f FLOP/clk/SM (status %d)\n",
                       where[a_in_tmem], n, issuers, per, 2.0 * 128 * n * 16 / per, st);
            }
    cudaFuncSetAttribute(mma_rate_layout, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    const char* layout_name[4] = {"128-byte swizzle", "64-byte swizzle", "32-byte swizzle", "no swizzle"};
    for (int a_in_tmem = 0; a_in_tmem < 2; ++a_in_tmem)
        for (int a_layout = 0; a_layout < (a_in_tmem ? 1 : 4); ++a_layout)
            for (int b_layout = 0; b_layout < 4; ++b_layout) {
                for (int rep = 0; rep < 2; ++rep) {
                    mma_rate_layout<<<sms, kThreads, kSmemBytes>>>(a_layout, b_layout, a_in_tmem, batches, out, status);
                    cudaError_t e = cudaDeviceSynchronize();
                    if (e != cudaSuccess) { printf("error %s\n", cudaGetErrorString(e)); return 1; }
                }
                unsigned long long cycles = 0;
                int st = 0;
                cudaMemcpy(&cycles, out, 8, cudaMemcpyDeviceToHost);
                cudaMemcpy(&st, status, 4, cudaMemcpyDeviceToHost);
                const double per = (double)cycles / (8.0 * batches);
                printf("layouts: A %s, B K-major %s, N = 128, 1 issuing thread: %6.1f cycles per MMA (status %d)\n",
                       a_in_tmem ? "in TMEM" : layout_name[a_layout], layout_name[b_layout], per, st);
            }
    cudaFuncSetAttribute(mma_rate_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    for (int a_in_tmem = 0; a_in_tmem < 2; ++a_in_tmem) {
        for (int rep = 0; rep < 2; ++rep) {
            mma_rate_pair<<<sms & ~1, kThreads, kSmemBytes>>>(a_in_tmem, batches, out, status);
            cudaError_t e = cudaDeviceSynchronize();
            if (e != cudaSuccess) { printf("error %s\n", cudaGetErrorString(e)); return 1; }
        }
        unsigned long long cycles = 0;
        int st = 0;
        cudaMemcpy(&cycles, out, 8, cudaMemcpyDeviceToHost);
        cudaMemcpy(&st, status, 4, cudaMemcpyDeviceToHost);
        const double per = (double)cycles / (8.0 * batches);
        printf("two SMs (cta_group::2), M = 256, N = 128, A in %s, 1 issuing thread: %6.1f cycles per MMA, %5.0f FLOP/clk/SM (status %d)\n",
               a_in_tmem ? "TMEM" : "smem", per, 2.0 * 128 * 128 * 16 / per, st);
    }
    return 0;
}
