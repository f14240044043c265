// Block-scaled MXFP4 GEMM on the 5th-generation tensor cores (the MXFP4 GEMM that replaces the
// linear layers' FP8 GEMM; operand orientation per Appendix C):
//   out[m][n] = alpha * sum_t 2^(sa[m][t]-127) 2^(sb[n][t]-127) sum_{k in block t} A[m][k] B[n][k]
//
// Persistent, warp-specialised, one CTA per SM, output tile 128 x 256:
//   warp 12      TMA producer: per K-step of 256 elements loads A (128 rows x 128 B of packed
//               codes) and B (256 rows x 128 B) in the 128-byte swizzle, plus the matching
//               scale tiles (512-byte blocks of 128 rows x 4 MX blocks), into a 4-stage ring.
//   warps 0..3   scale warps (one per TMEM lane quadrant): read each stage's scale tiles from
//                shared memory and write them into that stage's TMEM scale columns with
//                tcgen05.st.  (A tcgen05.cp would do the same copy, but each one occupies the
//                tensor pipe for about as long as an MMA and six are needed per stage.)
//   warps 4..11  epilogue: each warp pulls its 32 rows x 128 columns out of TMEM with four
//               back-to-back tcgen05.ld, hands the accumulator back to the MMA warp at once,
//               and only then scales by alpha, converts and stores (bf16 through a small
//               swizzled shared-memory staging buffer so that global stores are coalesced),
//               overlapping with the next tile's main loop.
//   warp 13      MMA issuer: four tcgen05.mma kind::mxf4.block_scale (K = 64 each) per stage;
//                the fp32 accumulator (128 lanes x 256 columns) lives in TMEM.
// Registers are rebalanced with setmaxnreg: the epilogue warps hold 128 accumulator values
// per thread, the other roles need few.  All waits are bounded (see ptx_sm100.cuh).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#ifdef MXFP4_PROBE
#include <stdlib.h>
#include <stdio.h>
#endif

#include "../../include/mxfp4.h"
#include "ptx_sm100.cuh"
#include "tma_host.cuh"

namespace mxfp4 {

constexpr int kGBlockM = 128;
constexpr int kGBlockN = 256;
constexpr int kGBlockK = 256;                    // elements per stage = 128 bytes of codes
constexpr int kGStages = 4;
constexpr int kGABytes = kGBlockM * 128;         // 16 KB
constexpr int kGBBytes = kGBlockN * 128;         // 32 KB
constexpr int kGSfaBytes = 2 * 512;              // 2 K-tiles of 128 elements
constexpr int kGSfbBytes = 2 * 2 * 512;          // 2 row blocks x 2 K-tiles
constexpr int kGEpiWarps = 8;
constexpr int kGProducerWarp = 12;
constexpr int kGMmaWarp = 13;
constexpr int kGThreads = 512;                   // 4 warpgroups: scales | epilogue x2 | producer+MMA
constexpr uint32_t kGTmemCols = 512;
constexpr uint32_t kGTmemSfBase = 256;           // accumulator occupies columns 0..255
constexpr uint32_t kGTmemSfPerBuf = 24;          // per stage: 8 columns SFA + 16 columns SFB

struct GemmSmem {
    alignas(1024) uint8_t a[kGStages][kGABytes];
    alignas(1024) uint8_t b[kGStages][kGBBytes];
    alignas(128) uint8_t sfa[kGStages][kGSfaBytes];
    alignas(128) uint8_t sfb[kGStages][kGSfbBytes];
    alignas(128) uint8_t out_stage[kGEpiWarps][32 * 64];   // 32 rows x 32 bf16 per warp
    alignas(8) uint64_t full[kGStages];
    uint64_t empty[kGStages];
    uint64_t sf_ready[kGStages];
    uint64_t tmem_full;
    uint64_t tmem_empty;
    uint32_t tmem_base;
    int abort_flag;
};

struct GemmParams {
    const uint8_t* a_scales;
    const uint8_t* b_scales;
    void* out;
    int64_t ld_out;
    int32_t M, N, K;
    int32_t tiles_m, tiles_n;
    int32_t k_stages;       // ceil(K / 256)
    int32_t sf_tiles_k;     // ceil(K / 128): 512-byte scale tiles per 128-row block
    int32_t sf_rows_b;      // ceil(N / 128)
    float alpha;
    int32_t out_fp32;
#ifdef MXFP4_PROBE
    int32_t debug;
    long long* probe_out;
#endif
};

// Instruction descriptor of tcgen05.mma kind::mxf4.block_scale: E2M1 x E2M1, E8M0 scales,
// both operands K-major, M = 128, N = 256.  Scale-factor ids select which byte pair of the
// 32-bit TMEM scale column an instruction uses.
__device__ __forceinline__ uint32_t make_idesc_mxf4(uint32_t a_sf_id, uint32_t b_sf_id)
{
    uint32_t d = 0;
    d |= b_sf_id << 4;                 // bits 4..5   B scale-factor id
    d |= 1u << 7;                      // bits 7..9   A format: E2M1
    d |= 1u << 10;                     // bits 10..12 B format: E2M1
    d |= (kGBlockN >> 3) << 17;        // bits 17..22 N / 8
    d |= 1u << 23;                     // bit 23      scale format: E8M0
    d |= (kGBlockM >> 4) << 24;        // bits 24..28 M / 16
    d |= a_sf_id << 29;                // bits 29..30 A scale-factor id
    return d;
}

__global__ void __launch_bounds__(kGThreads, 1)
gemm_mxf4_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                 const GemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    GemmSmem& sm = *reinterpret_cast<GemmSmem*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int total_tiles = p.tiles_m * p.tiles_n;
    const int my_tiles = blockIdx.x < total_tiles ? (total_tiles - 1 - blockIdx.x) / gridDim.x + 1 : 0;

    if (threadIdx.x == 0) {
        sm.abort_flag = 0;
        for (int s = 0; s < kGStages; ++s) {
            mbar_init(&sm.full[s], 1);
            mbar_init(&sm.empty[s], 1);
            mbar_init(&sm.sf_ready[s], 4);
        }
        mbar_init(&sm.tmem_full, 1);
        mbar_init(&sm.tmem_empty, kGEpiWarps);
        fence_barrier_init();
    }
    if (warp == kGMmaWarp) {
        tmem_alloc(&sm.tmem_base, kGTmemCols);
        tmem_relinquish();
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem = sm.tmem_base;
#ifdef MXFP4_PROBE
    long long pc0 = 0; unsigned long long pg0 = 0;
    if (threadIdx.x == 0 && blockIdx.x == 0) { pc0 = clock64(); asm volatile("mov.u64 %0, %globaltimer;" : "=l"(pg0)); }
#endif

    // register budget per role (whole warpgroups): 4*32*(56 + 2*192 + 56) = 63488 <= 65536;
    // every warp of a warpgroup executes the same setmaxnreg at the top of its role
    if (warp == kGProducerWarp) {
        // ------------------------------------------------------------ TMA producer
        setmaxnreg_dec<56>();
        if (lane == 0) {
            tma_prefetch_desc(&tm_a);
            tma_prefetch_desc(&tm_b);
            int it = 0;
            bool alive = true;
            for (int tile = blockIdx.x; alive && tile < total_tiles; tile += gridDim.x) {
                const int tm = tile % p.tiles_m, tn = tile / p.tiles_m;
                for (int ks = 0; ks < p.k_stages; ++ks, ++it) {
                    const int s = it % kGStages;
                    const uint32_t round = it / kGStages;
                    if (round > 0 && !mbar_wait(&sm.empty[s], (round - 1) & 1, &sm.abort_flag)) {
                        alive = false;
                        break;
                    }
                    const int kt0 = ks * 2;
                    const int nkt = min(2, p.sf_tiles_k - kt0);
                    const uint32_t sf_bytes = nkt * 512;
                    const int nb0 = tn * 2;
                    const int nnb = min(2, p.sf_rows_b - nb0);
                    mbar_arrive_expect_tx(&sm.full[s], kGABytes + kGBBytes + sf_bytes * (1 + nnb));
                    tma_load_2d(sm.a[s], &tm_a, &sm.full[s], ks * 128, tm * kGBlockM);
                    tma_load_2d(sm.b[s], &tm_b, &sm.full[s], ks * 128, tn * kGBlockN);
                    bulk_load_1d(sm.sfa[s], p.a_scales + (static_cast<int64_t>(tm) * p.sf_tiles_k + kt0) * 512,
                                 sf_bytes, &sm.full[s]);
                    for (int nb = 0; nb < nnb; ++nb)
                        bulk_load_1d(&sm.sfb[s][nb * 1024],
                                     p.b_scales + (static_cast<int64_t>(nb0 + nb) * p.sf_tiles_k + kt0) * 512,
                                     sf_bytes, &sm.full[s]);
                }
            }
        }
    } else if (warp == kGMmaWarp) {
        // ------------------------------------------------------------ MMA issuer
        setmaxnreg_dec<56>();
        if (lane == 0) {
            int it = 0;
            bool alive = true;
            for (int tile_it = 0; alive && tile_it < my_tiles; ++tile_it) {
#ifdef MXFP4_PROBE
                if (!(p.debug & 1))
#endif
                if (tile_it > 0 && !mbar_wait(&sm.tmem_empty, (tile_it - 1) & 1, &sm.abort_flag)) break;
                tcgen05_fence_after();
                for (int ks = 0; ks < p.k_stages; ++ks, ++it) {
                    const int s = it % kGStages;
                    const uint32_t parity = (it / kGStages) & 1;
                    // codes landed in shared memory, scales landed in this stage's TMEM columns
                    if (!mbar_wait(&sm.full[s], parity, &sm.abort_flag) ||
#ifdef MXFP4_PROBE
                        (!(p.debug & 2) && !mbar_wait(&sm.sf_ready[s], parity, &sm.abort_flag))) {
#else
                        !mbar_wait(&sm.sf_ready[s], parity, &sm.abort_flag)) {
#endif
                        alive = false;
                        break;
                    }
                    tcgen05_fence_after();
                    const uint32_t sf_tmem = tmem + kGTmemSfBase + s * kGTmemSfPerBuf;
                    const int valid_k = min(kGBlockK, p.K - ks * kGBlockK);
                    const int nmma = (valid_k + 63) / 64;
                    const uint64_t a_desc = make_smem_desc(smem_u32(sm.a[s]), 16, 1024, 2);
                    const uint64_t b_desc = make_smem_desc(smem_u32(sm.b[s]), 16, 1024, 2);
                    for (int j = 0; j < nmma; ++j) {
                        const uint32_t sf_id = (j & 1) * 2;
                        tcgen05_mma_mxf4(tmem, a_desc + 2 * j, b_desc + 2 * j,
                                         make_idesc_mxf4(sf_id, sf_id), sf_tmem + (j >> 1) * 4,
                                         sf_tmem + 8 + (j >> 1) * 8, (ks > 0 || j > 0) ? 1u : 0u);
                    }
                    // frees the shared-memory stage and its TMEM scale columns together
                    tcgen05_commit(&sm.empty[s]);
                }
                if (alive) tcgen05_commit(&sm.tmem_full);
            }
        }
    } else if (warp < 4) {
        // ------------------------------------------------------------ scale warps
        // Lane r of every quadrant must hold, per 128-row x 4-block scale tile, the 16 bytes at
        // offset 16*r of that tile: four 32-bit columns = rows r, r+32, r+64, r+96.  Stage s
        // owns TMEM columns [s*24, s*24+24): SFA K-tiles 0,1 | SFB K-tile 0 (row blocks 0,1) |
        // SFB K-tile 1.  The columns are free again once the producer has seen empty[s], which
        // happens before full[s] can complete, so waiting on full[s] is enough.
        setmaxnreg_dec<56>();
        const int total_it = my_tiles * p.k_stages;
        const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
        for (int it = 0; it < total_it; ++it) {
            const int s = it % kGStages;
            if (!mbar_wait(&sm.full[s], (it / kGStages) & 1, &sm.abort_flag)) break;
            const uint4 a0 = *reinterpret_cast<const uint4*>(&sm.sfa[s][lane * 16]);
            const uint4 a1 = *reinterpret_cast<const uint4*>(&sm.sfa[s][512 + lane * 16]);
            const uint4 b00 = *reinterpret_cast<const uint4*>(&sm.sfb[s][lane * 16]);
            const uint4 b01 = *reinterpret_cast<const uint4*>(&sm.sfb[s][1024 + lane * 16]);
            const uint4 b10 = *reinterpret_cast<const uint4*>(&sm.sfb[s][512 + lane * 16]);
            const uint4 b11 = *reinterpret_cast<const uint4*>(&sm.sfb[s][1536 + lane * 16]);
            const uint32_t t = tmem + lane_base + kGTmemSfBase + s * kGTmemSfPerBuf;
            tmem_st_32x32b_x8(t, a0, a1);
            tmem_st_32x32b_x8(t + 8, b00, b01);
            tmem_st_32x32b_x8(t + 16, b10, b11);
            tmem_st_wait();
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.sf_ready[s]);
        }
    } else if (warp < 12) {
        // ------------------------------------------------------------ epilogue warps
        setmaxnreg_inc<192>();
        const int ew = warp - 4;
        const int quad = warp & 3;                 // TMEM lane quadrant this warp may read
        const int half = ew >> 2;                  // which 128 accumulator columns
        uint8_t* stg = sm.out_stage[ew];
        int tile_it = 0;
        for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++tile_it) {
            const int tm = tile % p.tiles_m, tn = tile / p.tiles_m;
            if (!mbar_wait(&sm.tmem_full, tile_it & 1, &sm.abort_flag)) break;
            tcgen05_fence_after();
            uint32_t r[4][32];
            const uint32_t taddr = tmem + (static_cast<uint32_t>(quad * 32) << 16) + half * 128;
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld_32x32b_x32(taddr + c * 32, r[c]);
            tmem_ld_wait();
            // the accumulator is in registers: release TMEM before converting and storing
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.tmem_empty);

            const int64_t row0 = static_cast<int64_t>(tm) * kGBlockM + quad * 32;
            const int64_t colbase = static_cast<int64_t>(tn) * kGBlockN + half * 128;
            if (p.out_fp32) {
                const int64_t row = row0 + lane;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int64_t col0 = colbase + c * 32;
                    if (row >= p.M || col0 >= p.N) continue;
                    float* dst = static_cast<float*>(p.out) + row * p.ld_out + col0;
                    if (col0 + 32 <= p.N) {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            reinterpret_cast<float4*>(dst)[i] =
                                make_float4(__uint_as_float(r[c][4 * i]) * p.alpha,
                                            __uint_as_float(r[c][4 * i + 1]) * p.alpha,
                                            __uint_as_float(r[c][4 * i + 2]) * p.alpha,
                                            __uint_as_float(r[c][4 * i + 3]) * p.alpha);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (col0 + i < p.N) dst[i] = __uint_as_float(r[c][i]) * p.alpha;
                    }
                }
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    // own row (= lane), 32 columns -> 64 bytes, 16-byte chunk q stored at
                    // q ^ ((lane >> 1) & 3) so that both the row-wise writes and the
                    // 8-rows-per-instruction reads below are bank-conflict free
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint32_t w[4];
#pragma unroll
                        for (int h = 0; h < 4; ++h) {
                            const __nv_bfloat162 v = __floats2bfloat162_rn(
                                __uint_as_float(r[c][8 * q + 2 * h]) * p.alpha,
                                __uint_as_float(r[c][8 * q + 2 * h + 1]) * p.alpha);
                            w[h] = *reinterpret_cast<const uint32_t*>(&v);
                        }
                        *reinterpret_cast<uint4*>(stg + lane * 64 + ((q ^ ((lane >> 1) & 3)) * 16)) =
                            make_uint4(w[0], w[1], w[2], w[3]);
                    }
                    __syncwarp();
                    const int64_t col0 = colbase + c * 32 + (lane & 3) * 8;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int rr = i * 8 + (lane >> 2);
                        const uint4 v = *reinterpret_cast<const uint4*>(
                            stg + rr * 64 + (((lane & 3) ^ ((rr >> 1) & 3)) * 16));
                        const int64_t row = row0 + rr;
                        if (row < p.M && col0 < p.N) {
                            __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(p.out) + row * p.ld_out + col0;
                            if (col0 + 8 <= p.N) {
                                *reinterpret_cast<uint4*>(dst) = v;
                            } else {
                                const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&v);
                                for (int k = 0; k < 8; ++k)
                                    if (col0 + k < p.N) dst[k] = e[k];
                            }
                        }
                    }
                    __syncwarp();
                }
            }
        }
    }

    else {
        setmaxnreg_dec<56>();   // idle warps of the producer/MMA warpgroup
    }

    tcgen05_fence_before();
    __syncthreads();
#ifdef MXFP4_PROBE
    if (threadIdx.x == 0 && blockIdx.x == 0) { unsigned long long g1; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(g1)); p.probe_out[0] = clock64() - pc0; p.probe_out[1] = (long long)(g1 - pg0); }
#endif
    if (warp == kGMmaWarp) {
        tcgen05_fence_after();
        tmem_dealloc(tmem, kGTmemCols);
    }
}

static int launch_gemm(const void* a_codes, const void* a_scales, const void* b_codes,
                       const void* b_scales, int64_t M, int64_t N, int64_t K, float alpha, void* out,
                       int out_dtype, int64_t ld_out, int sm_count, cudaStream_t stream)
{
    CUtensorMap tm_a, tm_b;
    // codes as bytes: [rows x K/2], box = 128 bytes x (128 | 256) rows, 128-byte swizzle
    if (!make_tmap_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a_codes, M, K / 2, K / 2, kGBlockM, 128,
                      CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, b_codes, N, K / 2, K / 2, kGBlockN, 128,
                      CU_TENSOR_MAP_SWIZZLE_128B))
        return MXFP4_ERR_CUDA;
    GemmParams p;
    p.a_scales = static_cast<const uint8_t*>(a_scales);
    p.b_scales = static_cast<const uint8_t*>(b_scales);
    p.out = out;
    p.ld_out = ld_out;
    p.M = static_cast<int32_t>(M);
    p.N = static_cast<int32_t>(N);
    p.K = static_cast<int32_t>(K);
    p.tiles_m = static_cast<int32_t>((M + kGBlockM - 1) / kGBlockM);
    p.tiles_n = static_cast<int32_t>((N + kGBlockN - 1) / kGBlockN);
    p.k_stages = static_cast<int32_t>((K + kGBlockK - 1) / kGBlockK);
    p.sf_tiles_k = static_cast<int32_t>((K + 127) / 128);
    p.sf_rows_b = static_cast<int32_t>((N + 127) / 128);
    p.alpha = alpha;
    p.out_fp32 = out_dtype == MXFP4_OUT_FP32;
#ifdef MXFP4_PROBE
    { const char* e = getenv("MXFP4_GEMM_DEBUG"); p.debug = e ? atoi(e) : 0; static long long* buf = nullptr; if (!buf) cudaMalloc(&buf, 64); p.probe_out = buf; }
#endif
    const int64_t total = static_cast<int64_t>(p.tiles_m) * p.tiles_n;
    if (total > 0x7FFFFFFF) return MXFP4_ERR_SHAPE;
    const size_t smem = sizeof(GemmSmem) + 1024;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(gemm_mxf4_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem)) != cudaSuccess)
            return MXFP4_ERR_CUDA;
        attr_set = true;
    }
    const int grid = static_cast<int>(total < sm_count ? total : sm_count);
    gemm_mxf4_kernel<<<grid, kGThreads, smem, stream>>>(tm_a, tm_b, p);
#ifdef MXFP4_PROBE
    if (getenv("MXFP4_GEMM_CLOCK")) { long long h[2]; cudaStreamSynchronize(stream); cudaMemcpy(h, p.probe_out, 16, cudaMemcpyDeviceToHost); fprintf(stderr, "probe: %lld cycles in %lld ns -> %.0f MHz\n", h[0], h[1], h[0] * 1e3 / h[1]); }
#endif
    return cudaGetLastError() == cudaSuccess ? MXFP4_OK : MXFP4_ERR_CUDA;
}

}  // namespace mxfp4
