// Measuring aid: host time of one attn_fwd call made from C (argument checks, cached tensor maps, kernel launch), without
// the ctypes marshalling that bench.py's `host_call_us` includes.  A small shape whose kernel is short, twenty calls
// between two clock readings, the median of twenty such batches.
//
//     nvcc -O2 -std=c++17 -o profile_host_call profile_host_call.cu -Lpaper_2601_16032_b200 -lsawtooth_attn \
//         -Xlinker -rpath -Xlinker '$ORIGIN/paper_2601_16032_b200' && ./profile_host_call
#include <algorithm>
#include <chrono>
#include <cstdio>
#include <vector>

#include <cuda_runtime.h>

#include "include/sawtooth_attn.h"

int main() {
    const int N = 256, d = 64;
    void *q = nullptr, *o = nullptr;
    if (cudaMalloc(&q, (size_t)N * d * 2) != cudaSuccess || cudaMalloc(&o, (size_t)N * d * 2) != cudaSuccess) {
        printf("no CUDA device\n");
        return 1;
    }
    cudaMemset(q, 0, (size_t)N * d * 2);
    for (int i = 0; i < 20; ++i)
        if (attn_fwd(q, q, q, o, 1, 1, N, d, 0.125f, 0, ATTN_SCAN_SAWTOOTH, ATTN_F16, nullptr) != ATTN_OK) {
            printf("attn_fwd failed: %s\n", attn_last_error());
            return 1;
        }
    cudaDeviceSynchronize();
    std::vector<double> us;
    for (int r = 0; r < 20; ++r) {
        const auto t0 = std::chrono::steady_clock::now();
        for (int i = 0; i < 20; ++i) attn_fwd(q, q, q, o, 1, 1, N, d, 0.125f, 0, ATTN_SCAN_SAWTOOTH, ATTN_F16, nullptr);
        const auto t1 = std::chrono::steady_clock::now();
        us.push_back(std::chrono::duration<double, std::micro>(t1 - t0).count() / 20);
        cudaDeviceSynchronize();
    }
    std::sort(us.begin(), us.end());
    int code = 0;
    const int status = attn_device_status(&code);
    printf("attn_fwd from C: median %.2f us per call, fastest batch %.2f us (device status %d)\n", us[us.size() / 2], us[0], status);
    cudaFree(q);
    cudaFree(o);
    return status == ATTN_OK ? 0 : 1;
}
