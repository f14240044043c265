// Block-scaled MXFP4 GEMM, CTA-pair version (tcgen05 cta_group::2): two CTAs of a cluster share
// one 256 x 256 output tile.  Each CTA loads its own 128 rows of A and its own 128 rows of B per
// K-step (32 KB instead of the 48 KB a lone 128 x 256 tile needs), which is what matters once the
// L2 -> shared-memory operand feed, not the tensor pipe, bounds the kernel.  No TMA multicast is
// used: every CTA fetches its own operands; only barrier signals cross the pair.
//
//   out[m][n] = alpha * sum_t 2^(sa[m][t]-127) 2^(sb[n][t]-127) sum_{k in block t} A[m][k] B[n][k]
//
// Roles per CTA (512 threads, four warpgroups; same split as the single-CTA kernel):
//   warps 0..3   scale warps: shared memory -> this CTA's TMEM scale columns (tcgen05.st)
//   warps 4..11  epilogue: this CTA's 128 rows x 256 columns of the accumulator
//   warp 12      TMA producer: A half, B half (completion counted on the LEADER's barrier),
//                scale tiles (local barrier)
//   warp 13      MMA issuer -- only in the leader CTA (cluster rank 0); its commits arrive on
//                the barriers of both CTAs
// Barrier ownership: full / sf_ready / tmem_empty are consumed by the leader's MMA thread, so
// the peer's producers, scale warps and epilogue warps arrive on the leader's copies; empty and
// tmem_full are signalled in both CTAs by a multicast tcgen05.commit; sf_full is local.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#ifdef MXFP4_PROBE
#include <stdio.h>
#include <stdlib.h>
#endif

#include "../../include/mxfp4.h"
#include "ptx_sm100.cuh"
#include "tma_host.cuh"

namespace mxfp4 {

constexpr int kPHalfM = 128;                     // rows of A (and of the accumulator) per CTA
constexpr int kPHalfN = 128;                     // rows of B per CTA
constexpr int kPTileM = 256;
constexpr int kPTileN = 256;
constexpr int kPBlockK = 256;                    // elements per stage = 128 bytes of codes
constexpr int kPStages = 5;
constexpr int kPABytes = kPHalfM * 128;          // 16 KB
constexpr int kPBBytes = kPHalfN * 128;          // 16 KB
constexpr int kPSfaBytes = 2 * 512;              // own 128 rows x 2 K-tiles
constexpr int kPSfbBytes = 2 * 2 * 512;          // both 128-row blocks of B x 2 K-tiles
constexpr int kPEpiWarps = 8;
constexpr int kPProducerWarp = 12;
constexpr int kPMmaWarp = 13;
constexpr int kPThreads = 512;
constexpr uint32_t kPTmemCols = 512;
constexpr uint32_t kPTmemSfBase = 256;
constexpr uint32_t kPTmemSfPerBuf = 24;

struct GemmPairSmem {
    alignas(1024) uint8_t a[kPStages][kPABytes];
    alignas(1024) uint8_t b[kPStages][kPBBytes];
    alignas(128) uint8_t sfa[kPStages][kPSfaBytes];
    alignas(128) uint8_t sfb[kPStages][kPSfbBytes];
    alignas(128) uint8_t out_stage[kPEpiWarps][32 * 64];
    alignas(8) uint64_t full[kPStages];      // leader's copy is the live one
    uint64_t sf_full[kPStages];              // local
    uint64_t sf_ready[kPStages];             // leader's copy is the live one
    uint64_t empty[kPStages];                // both, via multicast commit
    uint64_t tmem_full;                      // both, via multicast commit
    uint64_t tmem_empty;                     // leader's copy is the live one
    uint32_t tmem_base;
    int abort_flag;
};

struct GemmPairParams {
    const uint8_t* a_scales;
    const uint8_t* b_scales;
    void* out;
    int64_t ld_out;
    int32_t M, N, K;
    int32_t tiles_m, tiles_n;   // 256 x 256 pair tiles
    int32_t k_stages;
    int32_t sf_tiles_k;         // ceil(K / 128)
    int32_t sf_rows_a;          // ceil(M / 128)
    int32_t sf_rows_b;          // ceil(N / 128)
    float alpha;
    int32_t out_fp32;
#ifdef MXFP4_PROBE
    long long* probe_out;
    int32_t debug;
#endif
};

// Instruction descriptor for the pair MMA: M = 256 (128 per CTA), N = 256.
__device__ __forceinline__ uint32_t make_idesc_mxf4_pair(uint32_t a_sf_id, uint32_t b_sf_id)
{
    uint32_t d = 0;
    d |= b_sf_id << 4;
    d |= 1u << 7;                      // A format E2M1
    d |= 1u << 10;                     // B format E2M1
    d |= (kPTileN >> 3) << 17;         // N / 8
    d |= 1u << 23;                     // scale format E8M0
    d |= (kPTileM >> 4) << 24;         // M / 16
    d |= a_sf_id << 29;
    return d;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPThreads, 1)
gemm_mxf4_pair_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                      const GemmPairParams p)
{
    extern __shared__ uint8_t smem_raw[];
    GemmPairSmem& sm = *reinterpret_cast<GemmPairSmem*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int cluster_id = blockIdx.x >> 1;
    const int n_clusters = gridDim.x >> 1;
    const int total_tiles = p.tiles_m * p.tiles_n;
    const int my_tiles = cluster_id < total_tiles ? (total_tiles - 1 - cluster_id) / n_clusters + 1 : 0;
    const int total_it = my_tiles * p.k_stages;

    if (threadIdx.x == 0) {
        sm.abort_flag = 0;
        for (int s = 0; s < kPStages; ++s) {
            mbar_init(&sm.full[s], 2);                 // one arrive.expect_tx per CTA
            mbar_init(&sm.sf_full[s], 1);
            mbar_init(&sm.sf_ready[s], 8);             // 4 scale warps x 2 CTAs
            mbar_init(&sm.empty[s], 1);
        }
        mbar_init(&sm.tmem_full, 1);
        mbar_init(&sm.tmem_empty, 2 * kPEpiWarps);
        fence_barrier_init();
    }
    if (warp == kPMmaWarp) {
        tmem_alloc_pair(&sm.tmem_base, kPTmemCols);
        tmem_relinquish_pair();
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();           // both CTAs' barriers exist before anyone signals across the pair
    tcgen05_fence_after();
    const uint32_t tmem = sm.tmem_base;

    if (warp == kPProducerWarp) {
        // ------------------------------------------------------------ TMA producer
        setmaxnreg_dec<56>();
        {
            // the whole warp walks the loop (uniform control flow keeps addresses and
            // descriptors in uniform registers); one elected lane issues the copies
            if (lane == 0) {
                tma_prefetch_desc(&tm_a);
                tma_prefetch_desc(&tm_b);
            }
            int it = 0;
            bool alive = true;
            for (int t = 0; alive && t < my_tiles; ++t) {
                const int tile = cluster_id + t * n_clusters;
                const int tm = tile % p.tiles_m, tn = tile / p.tiles_m;
                const int a_row_tile = tm * 2 + static_cast<int>(rank);     // 128-row scale tile of A
                for (int ks = 0; ks < p.k_stages; ++ks, ++it) {
                    const int s = it % kPStages;
                    const uint32_t round = it / kPStages;
                    if (round > 0 && !mbar_wait(&sm.empty[s], (round - 1) & 1, &sm.abort_flag)) {
                        alive = false;
                        break;
                    }
                    if (elect_one_sync()) {
                    // codes: counted on the leader's full barrier
                    const uint32_t full_leader = map_to_cta(smem_u32(&sm.full[s]), 0);
                    mbar_arrive_expect_tx_cluster(full_leader, kPABytes + kPBBytes);
                    tma_load_2d_pair(sm.a[s], &tm_a, full_leader, ks * 128, tm * kPTileM + rank * kPHalfM);
                    tma_load_2d_pair(sm.b[s], &tm_b, full_leader, ks * 128, tn * kPTileN + rank * kPHalfN);
                    // scales: local
                    const int kt0 = ks * 2;
                    const int nkt = min(2, p.sf_tiles_k - kt0);
                    const uint32_t sf_bytes = nkt * 512;
                    const int has_a = a_row_tile < p.sf_rows_a ? 1 : 0;
                    const int nb0 = tn * 2;
                    const int nnb = max(0, min(2, p.sf_rows_b - nb0));
                    mbar_arrive_expect_tx(&sm.sf_full[s], sf_bytes * (has_a + nnb));
                    if (has_a)
                        bulk_load_1d(sm.sfa[s],
                                     p.a_scales + (static_cast<int64_t>(a_row_tile) * p.sf_tiles_k + kt0) * 512,
                                     sf_bytes, &sm.sf_full[s]);
                    for (int nb = 0; nb < nnb; ++nb)
                        bulk_load_1d(&sm.sfb[s][nb * 1024],
                                     p.b_scales + (static_cast<int64_t>(nb0 + nb) * p.sf_tiles_k + kt0) * 512,
                                     sf_bytes, &sm.sf_full[s]);
                    }
                    __syncwarp();
                }
            }
        }
    } else if (warp == kPMmaWarp) {
        // ------------------------------------------------------------ MMA issuer (leader only)
        setmaxnreg_dec<56>();
        if (rank == 0) {
            // whole warp in uniform control flow; one elected lane issues MMAs and commits
            int it = 0;
            bool alive = true;
            for (int tile_it = 0; alive && tile_it < my_tiles; ++tile_it) {
                if (tile_it > 0 && !mbar_wait(&sm.tmem_empty, (tile_it - 1) & 1, &sm.abort_flag)) break;
                tcgen05_fence_after();
                for (int ks = 0; ks < p.k_stages; ++ks, ++it) {
                    const int s = it % kPStages;
                    const uint32_t parity = (it / kPStages) & 1;
#ifdef MXFP4_PROBE
                    long long pt0 = clock64();
                    bool okw = mbar_wait(&sm.full[s], parity, &sm.abort_flag);
                    long long pt1 = clock64();
                    okw = okw && ((p.debug & 2) || mbar_wait(&sm.sf_ready[s], parity, &sm.abort_flag));
                    long long pt2 = clock64();
                    if (blockIdx.x == 0 && it >= 64 && it < 128) {
                        p.probe_out[8 + (it - 64) * 3] = pt0; p.probe_out[8 + (it - 64) * 3 + 1] = pt1; p.probe_out[8 + (it - 64) * 3 + 2] = pt2;
                    }
                    if (!okw) { alive = false; break; }
#else
                    if (!mbar_wait(&sm.full[s], parity, &sm.abort_flag) ||
                        !mbar_wait(&sm.sf_ready[s], parity, &sm.abort_flag)) {
                        alive = false;
                        break;
                    }
#endif
                    tcgen05_fence_after();
                    const uint32_t sf_tmem = tmem + kPTmemSfBase + s * kPTmemSfPerBuf;
                    const int valid_k = min(kPBlockK, p.K - ks * kPBlockK);
                    const int nmma = (valid_k + 63) / 64;
                    const uint64_t a_desc = make_smem_desc(smem_u32(sm.a[s]), 16, 1024, 2);
                    const uint64_t b_desc = make_smem_desc(smem_u32(sm.b[s]), 16, 1024, 2);
                    if (elect_one_sync()) {
                    for (int j = 0; j < nmma; ++j) {
                        const uint32_t sf_id = (j & 1) * 2;
                        tcgen05_mma_mxf4_pair(tmem, a_desc + 2 * j, b_desc + 2 * j,
                                              make_idesc_mxf4_pair(sf_id, sf_id), sf_tmem + (j >> 1) * 4,
                                              sf_tmem + 8 + (j >> 1) * 8, (ks > 0 || j > 0) ? 1u : 0u);
#ifdef MXFP4_PROBE
                        if (blockIdx.x == 0 && it >= 64 && it < 128) p.probe_out[600 + (it - 64) * 5 + j] = clock64();
#endif
                    }
                    tcgen05_commit_pair(&sm.empty[s], 3);     // stage + scale columns free, both CTAs
#ifdef MXFP4_PROBE
                    if (blockIdx.x == 0 && it >= 64 && it < 128) p.probe_out[600 + (it - 64) * 5 + 4] = clock64();
#endif
                    }
                    __syncwarp();
                }
                __syncwarp();
                if (alive && elect_one_sync()) tcgen05_commit_pair(&sm.tmem_full, 3);
                __syncwarp();
            }
        }
    } else if (warp < 4) {
        // ------------------------------------------------------------ scale warps
        setmaxnreg_dec<56>();
        const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
#ifdef MXFP4_PROBE
        if (!(p.debug & 8))
#endif
        for (int it = 0; it < total_it; ++it) {
            const int s = it % kPStages;
#ifdef MXFP4_PROBE
            long long q0 = clock64();
#endif
            if (!mbar_wait(&sm.sf_full[s], (it / kPStages) & 1, &sm.abort_flag)) break;
#ifdef MXFP4_PROBE
            long long q1 = clock64();
#endif
            const uint4 a0 = *reinterpret_cast<const uint4*>(&sm.sfa[s][lane * 16]);
            const uint4 a1 = *reinterpret_cast<const uint4*>(&sm.sfa[s][512 + lane * 16]);
            const uint4 b00 = *reinterpret_cast<const uint4*>(&sm.sfb[s][lane * 16]);
            const uint4 b01 = *reinterpret_cast<const uint4*>(&sm.sfb[s][1024 + lane * 16]);
            const uint4 b10 = *reinterpret_cast<const uint4*>(&sm.sfb[s][512 + lane * 16]);
            const uint4 b11 = *reinterpret_cast<const uint4*>(&sm.sfb[s][1536 + lane * 16]);
            const uint32_t t = tmem + lane_base + kPTmemSfBase + s * kPTmemSfPerBuf;
            tmem_st_32x32b_x8(t, a0, a1);
            tmem_st_32x32b_x8(t + 8, b00, b01);
            tmem_st_32x32b_x8(t + 16, b10, b11);
#ifdef MXFP4_PROBE
            long long q2 = clock64();
#endif
            tmem_st_wait();
#ifdef MXFP4_PROBE
            long long q3 = clock64();
#endif
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&sm.sf_ready[s]), 0));
#ifdef MXFP4_PROBE
            if (blockIdx.x == 0 && warp == 0 && lane == 0 && it >= 64 && it < 128) {
                long long q4 = clock64();
                long long* o = p.probe_out + 256 + (it - 64) * 5;
                o[0] = q0; o[1] = q1; o[2] = q2; o[3] = q3; o[4] = q4;
            }
#endif
        }
    } else if (warp < 12) {
        // ------------------------------------------------------------ epilogue warps
        setmaxnreg_inc<192>();
        const int ew = warp - 4;
        const int quad = warp & 3;
        const int half = ew >> 2;
        uint8_t* stg = sm.out_stage[ew];
        const uint32_t tmem_empty_leader = map_to_cta(smem_u32(&sm.tmem_empty), 0);
        for (int tile_it = 0; tile_it < my_tiles; ++tile_it) {
            const int tile = cluster_id + tile_it * n_clusters;
            const int tm = tile % p.tiles_m, tn = tile / p.tiles_m;
            if (!mbar_wait(&sm.tmem_full, tile_it & 1, &sm.abort_flag)) break;
            tcgen05_fence_after();
            uint32_t r[4][32];
            const uint32_t taddr = tmem + (static_cast<uint32_t>(quad * 32) << 16) + half * 128;
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld_32x32b_x32(taddr + c * 32, r[c]);
            tmem_ld_wait();
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(tmem_empty_leader);

            const int64_t row0 = static_cast<int64_t>(tm) * kPTileM + rank * kPHalfM + quad * 32;
            const int64_t colbase = static_cast<int64_t>(tn) * kPTileN + half * 128;
#ifdef MXFP4_PROBE
            if (p.debug & 4) continue;
#endif
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
    } else {
        setmaxnreg_dec<56>();   // idle warps of the producer/MMA warpgroup
    }

    // neither CTA may leave (or free TMEM) while its peer can still signal it or read its memory
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == kPMmaWarp) {
        tcgen05_fence_after();
        tmem_dealloc_pair(tmem, kPTmemCols);
    }
}

static int launch_gemm_pair(const void* a_codes, const void* a_scales, const void* b_codes,
                            const void* b_scales, int64_t M, int64_t N, int64_t K, float alpha, void* out,
                            int out_dtype, int64_t ld_out, int sm_count, cudaStream_t stream)
{
    CUtensorMap tm_a, tm_b;
    if (!make_tmap_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a_codes, M, K / 2, K / 2, kPHalfM, 128,
                      CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, b_codes, N, K / 2, K / 2, kPHalfN, 128,
                      CU_TENSOR_MAP_SWIZZLE_128B))
        return MXFP4_ERR_CUDA;
    GemmPairParams p;
    p.a_scales = static_cast<const uint8_t*>(a_scales);
    p.b_scales = static_cast<const uint8_t*>(b_scales);
    p.out = out;
    p.ld_out = ld_out;
    p.M = static_cast<int32_t>(M);
    p.N = static_cast<int32_t>(N);
    p.K = static_cast<int32_t>(K);
    p.tiles_m = static_cast<int32_t>((M + kPTileM - 1) / kPTileM);
    p.tiles_n = static_cast<int32_t>((N + kPTileN - 1) / kPTileN);
    p.k_stages = static_cast<int32_t>((K + kPBlockK - 1) / kPBlockK);
    p.sf_tiles_k = static_cast<int32_t>((K + 127) / 128);
    p.sf_rows_a = static_cast<int32_t>((M + 127) / 128);
    p.sf_rows_b = static_cast<int32_t>((N + 127) / 128);
    p.alpha = alpha;
    p.out_fp32 = out_dtype == MXFP4_OUT_FP32;
#ifdef MXFP4_PROBE
    { static long long* buf = nullptr; if (!buf) cudaMalloc(&buf, 8192); p.probe_out = buf; const char* e = getenv("MXFP4_GEMM_DEBUG"); p.debug = e ? atoi(e) : 0; }
#endif
    const int64_t total = static_cast<int64_t>(p.tiles_m) * p.tiles_n;
    if (total > 0x3FFFFFFF) return MXFP4_ERR_SHAPE;
    const size_t smem = sizeof(GemmPairSmem) + 1024;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(gemm_mxf4_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem)) != cudaSuccess)
            return MXFP4_ERR_CUDA;
        attr_set = true;
    }
    const int max_clusters = sm_count / 2;
    const int clusters = static_cast<int>(total < max_clusters ? total : max_clusters);
    gemm_mxf4_pair_kernel<<<2 * clusters, kPThreads, smem, stream>>>(tm_a, tm_b, p);
#ifdef MXFP4_PROBE
    if (getenv("MXFP4_GEMM_TRACE")) { static long long h[1024]; cudaStreamSynchronize(stream); cudaMemcpy(h, p.probe_out, 8192, cudaMemcpyDeviceToHost); for (int i = 1; i < 64; ++i) { long long* o = h + 256 + i * 5; fprintf(stderr, "scale it %d: loop gap %lld | wait sf_full %lld | lds+st issue %lld | wait::st %lld | arrive %lld\n", 64 + i, o[0] - o[-1], o[1] - o[0], o[2] - o[1], o[3] - o[2], o[4] - o[3]); } for (int i = 0; i < 64; ++i) { long long* o = h + 600 + i * 5; fprintf(stderr, "issue it %d: mma0 %lld mma1 %lld mma2 %lld mma3 %lld commit %lld\n", 64 + i, o[0] - h[8 + i * 3 + 2], o[1] - o[0], o[2] - o[1], o[3] - o[2], o[4] - o[3]); } for (int i = 0; i < 64; ++i) fprintf(stderr, "it %d: since prev issue %lld | wait full %lld | wait sf %lld\n", 64 + i, i ? h[8 + i * 3] - h[8 + (i - 1) * 3 + 2] : 0, h[8 + i * 3 + 1] - h[8 + i * 3], h[8 + i * 3 + 2] - h[8 + i * 3 + 1]); }
#endif
    return cudaGetLastError() == cudaSuccess ? MXFP4_OK : MXFP4_ERR_CUDA;
}

}  // namespace mxfp4
