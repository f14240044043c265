// Diagnostic kernel (no counterpart in the paper): the rate of the GEMM's pair MMA -- 256 x 192 x 64,
// kind::mxf4.block_scale, eight per iteration exactly as one K-step of gemm_mxf4_pair_kernel issues
// them -- on operands that never leave shared memory: no TMA, no L2 traffic, no epilogue.  What it
// measures is the ceiling the tensor pipe itself sets on this device for MXFP4, with constant
// operand bits (clock-bound) and with random ones (power-bound), i.e. the denominator against
// which the GEMM's operand movement, tile switches and epilogue can be read.
#pragma once

#include "gemm_pair_kernel.cuh"

namespace mxfp4 {

struct MmaProbeSmem {
    alignas(1024) uint8_t a[kPStages][kPABytes];
    alignas(1024) uint8_t b[kPStages][2][kPBSubBytes];
    alignas(8) uint64_t done;
    uint32_t tmem_base;
    int abort_flag;
};

constexpr int kMmaProbeThreads = 128;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kMmaProbeThreads, 1)
mma_rate_probe_kernel(int iterations, int random_operands)
{
    extern __shared__ uint8_t smem_raw[];
    MmaProbeSmem& sm = *reinterpret_cast<MmaProbeSmem*>(smem_align_1024(smem_raw));
    // operand bits: a constant pattern, or a per-thread linear congruential sequence
    uint32_t x = 1234567u + blockIdx.x * 7919u + threadIdx.x * 104729u;
    constexpr int kWords = (kPStages * kPABytes + kPStages * 2 * kPBSubBytes) / 4;
    for (int i = threadIdx.x; i < kWords; i += kMmaProbeThreads) {
        x = x * 1664525u + 1013904223u;
        reinterpret_cast<uint32_t*>(&sm)[i] = random_operands ? (x ^ (x >> 13)) : 0x22222222u;
    }
    if (threadIdx.x == 0) {
        sm.abort_flag = 0;
        mbar_init(&sm.done, 1);
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        tmem_alloc_pair(&sm.tmem_base, kPTmemCols);
        tmem_relinquish_pair();
    }
    fence_proxy_async_smem();
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();
    tcgen05_fence_after();
    const uint32_t tmem = sm.tmem_base;
    const uint32_t rank = cluster_ctarank();
    {
        // scale columns of all four stage slots: 2^0 (constant) or 2^-2 .. 2^1 (random)
        const uint32_t sv = random_operands ? (0x7d7d7d7du + ((x >> 8) & 0x03030303u)) : 0x7f7f7f7fu;
        const uint4 v = make_uint4(sv, sv, sv, sv);
        const uint32_t t = tmem + (static_cast<uint32_t>((threadIdx.x >> 5) * 32) << 16) + kPTmemSfBase;
        for (uint32_t c = 0; c < kPStages * kPTmemSfPerBuf; c += 8) tmem_st_32x32b_x8(t + c, v, v);
        tmem_st_wait();
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();
    tcgen05_fence_after();
    if (threadIdx.x < 32 && rank == 0) {
        const uint32_t idesc0 = make_idesc_mx_pair<0>(0, 0) | idesc_n(kPMmaN);
        const uint32_t idesc2 = make_idesc_mx_pair<0>(2, 2) | idesc_n(kPMmaN);
        for (int it = 0; it < iterations; ++it) {
            const int s = it % kPStages;
            if (elect_one_sync()) {
                const uint64_t a_desc = make_smem_desc(smem_u32(sm.a[s]), 16, 1024, 2);
                const uint64_t b_desc = make_smem_desc(smem_u32(sm.b[s][0]), 16, 1024, 2);
                const uint32_t sf = tmem + kPTmemSfBase + s * kPTmemSfPerBuf;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t idesc = (j & 1) ? idesc2 : idesc0;
                    const uint32_t sfa = sf + (j >> 1) * 4, sfb = sf + 8 + (j >> 1) * 12;
                    const uint32_t acc = (it > 0 || j > 0) ? 1u : 0u;
                    tcgen05_mma_mx_pair_collect<0, 0>(tmem, a_desc + 2 * j, b_desc + 2 * j, idesc, sfa, sfb, acc);
                    tcgen05_mma_mx_pair_collect<0, 1>(tmem + kPMmaN, a_desc + 2 * j, b_desc + 2 * j + (kPBSubBytes >> 4),
                                                      idesc, sfa, sfb + 6, acc);
                }
            }
            __syncwarp();
        }
        if (elect_one_sync()) tcgen05_commit_pair(&sm.done, 1);
        __syncwarp();
        mbar_wait(&sm.done, 0, &sm.abort_flag);      // bounded like every wait of the library
    }
    // neither CTA may leave (or free TMEM) while its peer can still use it
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (threadIdx.x < 32) {
        tcgen05_fence_after();
        tmem_dealloc_pair(tmem, kPTmemCols);
    }
}

}  // namespace mxfp4
