// Helpers shared by the dense-transform kernels (kernels_generic.cu, kernels_nd.cu): magnitude keys, a
// CTA-wide prefix sum, the exact radix select behind the top-k, and the persistent-grid launcher.
#pragma once

#include "demo_internal.h"

namespace {

constexpr int GEN_THREADS = 256;

__device__ __forceinline__ unsigned mag_key(float v) { return __float_as_uint(v) & 0x7fffffffu; }

// Exclusive prefix sum of one unsigned per thread over the 256-thread CTA.
__device__ __forceinline__ unsigned block_exclusive_scan(unsigned v, unsigned *warp_tot /*[8]*/)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        unsigned n = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += n;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    unsigned base = 0;
    for (int w = 0; w < warp; ++w) base += warp_tot[w];
    __syncthreads();
    return base + inc - v;
}

// Exact k-th largest magnitude of Q[0..M) by radix select on the fp32 magnitude bits (which order
// like the magnitudes).  Returns the key of the k-th largest in *thr and, in *need_eq, how many
// elements EQUAL to it belong to the top-k (those with the lowest indices are taken).
__device__ __forceinline__ void radix_select(const float *Q, int M, int k_eff, unsigned *hist, unsigned *s_state,
                                             unsigned *thr, unsigned *need_eq)
{
    const int tid = threadIdx.x;
    if (tid == 0) {
        s_state[0] = 0u;              // prefix of the key found so far
        s_state[1] = (unsigned)k_eff; // rank still to resolve inside the prefix class
    }
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        const unsigned mask = (pass == 0) ? 0u : (0xffffffffu << (shift + 8));
        hist[tid] = 0u;
        __syncthreads();
        const unsigned prefix = s_state[0];
        for (int i = tid; i < M; i += GEN_THREADS) {
            const unsigned key = mag_key(Q[i]);
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (tid < 32) {
            // lane l owns bins 255-8l ... 248-8l (descending magnitude)
            const unsigned rem = s_state[1];
            unsigned local = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) local += hist[255 - 8 * tid - j];
            unsigned inc = local;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                unsigned n = __shfl_up_sync(0xffffffffu, inc, d);
                if (tid >= d) inc += n;
            }
            const unsigned before = inc - local;
            if (before < rem && rem <= inc) {  // exactly one lane
                unsigned cum = before;
                int b = 255 - 8 * tid;
                for (int j = 0; j < 8; ++j, --b) {
                    const unsigned h = hist[b];
                    if (cum + h >= rem) break;
                    cum += h;
                }
                s_state[1] = rem - cum;
                s_state[0] = prefix | ((unsigned)b << shift);
            }
        }
        __syncthreads();
    }
    *thr = s_state[0];
    *need_eq = s_state[1];
    __syncthreads();
}

template <typename K>
cudaError_t launch_persistent(K kernel, size_t smem, long long n_chunks, int sm_count, cudaStream_t stream,
                              const void *args_struct_ptr)
{
    if (n_chunks <= 0) return cudaSuccess;
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    int per_sm = 0;
    err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, GEN_THREADS, smem);
    if (err != cudaSuccess) return err;
    if (per_sm < 1) per_sm = 1;
    long long grid = (long long)sm_count * per_sm;
    if (grid > n_chunks) grid = n_chunks;
    void *params[] = {const_cast<void *>(args_struct_ptr)};
    return cudaLaunchKernel((const void *)kernel, dim3((unsigned)grid), dim3(GEN_THREADS), params, smem, stream);
}

}  // namespace
