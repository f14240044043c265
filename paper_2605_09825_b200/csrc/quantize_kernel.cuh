// MXFP4 quantize kernel (Appendix A.1 Eq. (1), rotation of Appendix A.2, block orientation of
// Appendix D), one persistent CTA per SM.
//
// Work unit: a tile of 128 operand rows x 128 elements along K (4 MX blocks).  A producer warp
// streams source tiles into a ring of shared-memory stages with TMA; 512 consumer threads each
// own one 32-element block per tile: the whole block sits in the thread's registers, so the
// five butterfly stages, the block maximum and the rounding need no cross-lane traffic.
// Results leave through shared memory: packed codes as a 128 x 64-byte tile written by a TMA
// store (which also clips ragged edges), scales as one contiguous 512-byte tile.
//
//   AXIS 1 (row-wise blocks):    operand row = source row; a stage holds two 128-row x 64-col
//                                boxes in the 128-byte swizzle, read back 16 bytes at a time.
//   AXIS 0 (column-wise blocks): operand row = source column; a stage holds one 128 x 128 box,
//                                each thread walks 32 rows of one column.  The operand comes
//                                out transposed without a separate transpose pass.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx_sm100.cuh"

namespace mxfp4 {

constexpr int kQTileO = 128;                 // operand rows per tile
constexpr int kQTileK = 128;                 // elements along K per tile (4 blocks)
constexpr int kQStageBytes = 128 * 128 * 2;  // one source tile, bf16
constexpr int kQStages = 4;
constexpr int kQConsumers = 512;
constexpr int kQThreads = kQConsumers + 32;
constexpr int kQCodeTileBytes = 128 * 64;
constexpr int kQScaleTileBytes = 512;

struct QuantSmem {
    alignas(1024) uint8_t stage[kQStages][kQStageBytes];
    alignas(1024) uint8_t code_tile[2][kQCodeTileBytes];
    alignas(128) uint8_t scale_tile[2][kQScaleTileBytes];
    alignas(8) uint64_t full[kQStages];
    uint64_t empty[kQStages];
    int abort_flag;
};

struct QuantParams {
    uint8_t* scales;
    int64_t outer, K;        // operand view
    int64_t nt;              // K / 32
    int32_t tiles_o, tiles_k;
    uint32_t seed_lo, seed_hi, tag, sign_mask;
    int32_t scale_layout;    // 0 canonical, 1 tiled
};

// In-register 32-point Walsh-Hadamard transform, stages h = 1, 2, 4, 8, 16; every output is
// one fp32 add or subtract (no FMA contraction can occur: there are no multiplies).
__device__ __forceinline__ void fwht32(float (&v)[32])
{
#pragma unroll
    for (int h = 1; h < 32; h <<= 1) {
#pragma unroll
        for (int i = 0; i < 32; i += 2 * h) {
#pragma unroll
            for (int j = i; j < i + h; ++j) {
                const float a = v[j], b = v[j + h];
                v[j] = __fadd_rn(a, b);
                v[j + h] = __fsub_rn(a, b);
            }
        }
    }
}

// Two E2M1 codes from two floats, round-to-nearest-even, saturating: `lo` lands in bits 3:0.
__device__ __forceinline__ uint32_t cvt_e2m1x2(float lo, float hi)
{
    uint16_t r;
    asm("{\n\t.reg .b8 t;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 t, %1, %2;\n\t"
        "cvt.u16.u8 %0, t;\n\t}"
        : "=h"(r)
        : "f"(hi), "f"(lo));
    return r;
}

// Stochastic rounding of one scaled value with 8 random bits.  |s| * 2^-126 re-biases the value
// so that bits 22.. of its fp32 pattern are the E2M1 magnitude code below it and bits 0..21 the
// position between the two neighbouring grid points; rounding the product toward +inf keeps
// every strict comparison against the (integer) thresholds intact.
__device__ __forceinline__ uint32_t sr_e2m1(float s, uint32_t u8)
{
    const float a = fminf(fabsf(s), 6.0f);
    const uint32_t bits = __float_as_uint(__fmul_ru(a, 1.1754943508222875e-38f));
    const uint32_t r = bits + (0x3FFFFFu - ((2u * u8 + 1u) << 13));
    return (r >> 22) | ((__float_as_uint(s) >> 28) & 8u);
}

template <int AXIS, int HMODE, int SR>
__global__ void __launch_bounds__(kQThreads, 1)
quantize_kernel(const __grid_constant__ CUtensorMap tm_src, const __grid_constant__ CUtensorMap tm_codes,
                const QuantParams p)
{
    extern __shared__ uint8_t smem_raw[];
    QuantSmem& sm = *reinterpret_cast<QuantSmem*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int tid = threadIdx.x;
    const int total_tiles = p.tiles_o * p.tiles_k;

    if (tid == 0) {
        sm.abort_flag = 0;
        for (int s = 0; s < kQStages; ++s) {
            mbar_init(&sm.full[s], 1);
            mbar_init(&sm.empty[s], kQConsumers / 32);
        }
        fence_barrier_init();
    }
    __syncthreads();

    if (tid >= kQConsumers) {
        // ------------------------------------------------------------ producer warp
        if (tid == kQConsumers) {
            tma_prefetch_desc(&tm_src);
            int it = 0;
            for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++it) {
                const int s = it % kQStages;
                const uint32_t round = it / kQStages;
                if (round > 0 && !mbar_wait(&sm.empty[s], (round - 1) & 1, &sm.abort_flag)) break;
                // the fastest-varying tile index walks the source's contiguous axis
                int to, tk;
                if (AXIS == 1) { to = tile / p.tiles_k; tk = tile % p.tiles_k; }
                else           { tk = tile / p.tiles_o; to = tile % p.tiles_o; }
                mbar_arrive_expect_tx(&sm.full[s], kQStageBytes);
                if (AXIS == 1) {
                    tma_load_2d(&sm.stage[s][0], &tm_src, &sm.full[s], tk * kQTileK, to * kQTileO);
                    tma_load_2d(&sm.stage[s][kQStageBytes / 2], &tm_src, &sm.full[s],
                                tk * kQTileK + 64, to * kQTileO);
                } else {
                    tma_load_2d(&sm.stage[s][0], &tm_src, &sm.full[s], to * kQTileO, tk * kQTileK);
                }
            }
        }
        return;
    }

    // ---------------------------------------------------------------- consumers
    const int kb = tid >> 7;   // which of the tile's 4 blocks along K
    const int o = tid & 127;   // operand row inside the tile
    if (tid == 0) tma_prefetch_desc(&tm_codes);

    int it = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++it) {
        const int s = it % kQStages;
        const uint32_t round = it / kQStages;
        const int buf = it & 1;
        int to, tk;
        if (AXIS == 1) { to = tile / p.tiles_k; tk = tile % p.tiles_k; }
        else           { tk = tile / p.tiles_o; to = tile % p.tiles_o; }

        const bool ok = mbar_wait(&sm.full[s], round & 1, &sm.abort_flag);

        float v[32];
        if (ok) {
            if (AXIS == 1) {
                const uint8_t* base = &sm.stage[s][(kb >> 1) * (kQStageBytes / 2) + o * 128];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int chunk = (((kb & 1) * 4 + j) ^ (o & 7)) * 16;
                    const uint4 q = *reinterpret_cast<const uint4*>(base + chunk);
                    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        v[8 * j + 2 * i] = __uint_as_float(w[i] << 16);
                        v[8 * j + 2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
                    }
                }
            } else {
                const uint16_t* base =
                    reinterpret_cast<const uint16_t*>(&sm.stage[s][0]) + (kb * 32) * 128 + o;
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    v[j] = __uint_as_float(static_cast<uint32_t>(base[j * 128]) << 16);
            }
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = 0.0f;
        }
        // the stage is in registers now: hand it back to the producer
        __syncwarp();
        if ((tid & 31) == 0) mbar_arrive(&sm.empty[s]);

        if (HMODE == 2) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                v[j] = __uint_as_float(__float_as_uint(v[j]) ^ ((p.sign_mask << (31 - j)) & 0x80000000u));
        }
        if (HMODE != 0) fwht32(v);

        float amax = 0.0f;
#pragma unroll
        for (int j = 0; j < 32; ++j) amax = fmaxf(amax, fabsf(v[j]));
        const uint32_t E = __float_as_uint(amax) >> 23;
        const uint32_t byte = E > 2u ? E - 2u : 0u;   // E <= 255 keeps byte <= 253 < 255
        const float mult = __uint_as_float((254u - byte) << 23);

        uint32_t packed[4];
        if (SR == 0) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t w = 0;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float lo = __fmul_rn(v[8 * q + 2 * i], mult);
                    const float hi = __fmul_rn(v[8 * q + 2 * i + 1], mult);
                    w |= cvt_e2m1x2(lo, hi) << (8 * i);
                }
                packed[q] = w;
            }
        } else {
            const uint64_t e0 = static_cast<uint64_t>(to * kQTileO + o) * static_cast<uint64_t>(p.K) +
                                static_cast<uint64_t>((tk * 4 + kb) * 32);
            const uint64_t g = e0 >> 4;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t r[4];
                const uint64_t gg = g + half;
                philox4x32_10(static_cast<uint32_t>(gg), static_cast<uint32_t>(gg >> 32), p.tag, 0u,
                              p.seed_lo, p.seed_hi, r);
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    uint32_t w = 0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int j = half * 16 + q * 8 + i;       // element in the block
                        const int e = q * 8 + i;                   // element in the 16-group
                        const uint32_t u8 = (r[e >> 2] >> (8 * (e & 3))) & 0xFFu;
                        w |= sr_e2m1(__fmul_rn(v[j], mult), u8) << (4 * i);
                    }
                    packed[half * 2 + q] = w;
                }
            }
        }

        // stage the results: codes in the 64-byte swizzle the TMA store expects
        *reinterpret_cast<uint4*>(&sm.code_tile[buf][o * 64 + ((kb ^ ((o >> 1) & 3)) * 16)]) =
            make_uint4(packed[0], packed[1], packed[2], packed[3]);
        if (p.scale_layout == 1) {
            sm.scale_tile[buf][(o & 31) * 16 + (o >> 5) * 4 + kb] = static_cast<uint8_t>(byte);
        } else {
            const int64_t og = static_cast<int64_t>(to) * kQTileO + o;
            const int64_t tg = static_cast<int64_t>(tk) * 4 + kb;
            if (ok && og < p.outer && tg < p.nt) p.scales[og * p.nt + tg] = static_cast<uint8_t>(byte);
        }
        fence_proxy_async_smem();
        // the store issued one tile ago must have drained its buffer before the next tile
        // (which every thread reaches only through the barrier below) overwrites it
        if (tid == 0) bulk_wait_group_read<0>();
        uint32_t any_fail;
        asm volatile(
            "{\n\t.reg .pred P, Q;\n\t"
            "setp.ne.u32 Q, %1, 0;\n\t"
            "barrier.cta.red.or.pred P, 1, %2, Q;\n\t"
            "selp.u32 %0, 1, 0, P;\n\t}"
            : "=r"(any_fail)
            : "r"(ok ? 0u : 1u), "n"(kQConsumers)
            : "memory");
        if (any_fail) break;
        if (tid == 0) {
            tma_store_2d(&tm_codes, &sm.code_tile[buf][0], tk * (kQTileK / 2), to * kQTileO);
            if (p.scale_layout == 1)
                bulk_store_1d(p.scales + (static_cast<int64_t>(to) * p.tiles_k + tk) * kQScaleTileBytes,
                              &sm.scale_tile[buf][0], kQScaleTileBytes);
            bulk_commit_group();
        }
    }
    if (tid == 0) bulk_wait_group<0>();
}

}  // namespace mxfp4
