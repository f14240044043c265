// MXFP4 quantize kernel (Appendix A.1 Eq. (1), rotation of Appendix A.2, block orientation of
// Appendix D), one persistent CTA per SM.
//
// Work unit: a tile of 128 operand rows x 128 elements along K (4 MX blocks).  A producer warp
// streams source tiles into a ring of shared-memory stages with TMA; 512 consumer threads each
// own one 32-element block per tile: the whole block sits in the thread's registers, so the
// five butterfly stages (as packed fp32x2 operations), the block maximum and the rounding
// need no cross-lane traffic.
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

// Packed fp32 pairs: sm_100 adds, subtracts and multiplies two independent fp32 values held in
// one 64-bit register with a single instruction (each lane is an ordinary IEEE fp32
// round-to-nearest operation, so results are bit-identical to the scalar form).
__device__ __forceinline__ uint64_t pack2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}

__device__ __forceinline__ void unpack2(uint64_t p, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p));
}

__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// max(|a|, |b|, |c|) in one instruction.
__device__ __forceinline__ float max3_abs(float a, float b, float c)
{
    float r;
    asm("max.abs.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// In-register 32-point Walsh-Hadamard transform of v[0..31] held as 16 pairs
// P[i] = (v[2i], v[2i+1]).  Stage h = 1 was applied by the caller while forming the pairs
// (its partners share a pair); stages h = 2, 4, 8, 16 pair whole registers, so each packed
// add/sub does two butterflies.  Same five stages, same order, one fp32 rounding per output.
__device__ __forceinline__ void fwht32_stages_2_to_16(uint64_t (&P)[16])
{
#pragma unroll
    for (int hp = 1; hp < 16; hp <<= 1) {
#pragma unroll
        for (int i = 0; i < 16; i += 2 * hp) {
#pragma unroll
            for (int j = i; j < i + hp; ++j) {
                const uint64_t a = P[j], b = P[j + hp];
                P[j] = add2(a, b);
                P[j + hp] = sub2(a, b);
            }
        }
    }
}

// Eight E2M1 codes (one 32-bit word of packed output) from eight floats, round-to-nearest-even,
// saturating; v0 lands in bits 3:0, v7 in bits 31:28.
__device__ __forceinline__ uint32_t cvt_e2m1x8(float v0, float v1, float v2, float v3, float v4,
                                               float v5, float v6, float v7)
{
    uint32_t r;
    asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
        "mov.b32 %0, {b0, b1, b2, b3};\n\t}"
        : "=r"(r)
        : "f"(v0), "f"(v1), "f"(v2), "f"(v3), "f"(v4), "f"(v5), "f"(v6), "f"(v7));
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

        // the block as 16 packed pairs P[i] = (v[2i], v[2i+1]); the sign diagonal and the first
        // butterfly stage (whose partners are the two halves of a pair) are applied on the way in
        uint64_t P[16];
        auto make_pair = [&](int i, uint32_t lo_bits, uint32_t hi_bits) {
            if (HMODE == 2) {
                lo_bits ^= (p.sign_mask << (31 - 2 * i)) & 0x80000000u;
                hi_bits ^= (p.sign_mask << (30 - 2 * i)) & 0x80000000u;
            }
            const float a = __uint_as_float(lo_bits), b = __uint_as_float(hi_bits);
            P[i] = HMODE != 0 ? pack2(__fadd_rn(a, b), __fsub_rn(a, b)) : pack2(a, b);
        };
        if (ok) {
            if (AXIS == 1) {
                const uint8_t* base = &sm.stage[s][(kb >> 1) * (kQStageBytes / 2) + o * 128];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int chunk = (((kb & 1) * 4 + j) ^ (o & 7)) * 16;
                    const uint4 q = *reinterpret_cast<const uint4*>(base + chunk);
                    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) make_pair(4 * j + i, w[i] * 65536u, w[i] & 0xFFFF0000u);
                }
            } else {
                const uint16_t* base =
                    reinterpret_cast<const uint16_t*>(&sm.stage[s][0]) + (kb * 32) * 128 + o;
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    make_pair(i, static_cast<uint32_t>(base[(2 * i) * 128]) * 65536u,
                              static_cast<uint32_t>(base[(2 * i + 1) * 128]) * 65536u);
            }
        } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) P[i] = 0ull;
        }
        // the stage is in registers now: hand it back to the producer
        __syncwarp();
        if ((tid & 31) == 0) mbar_arrive(&sm.empty[s]);

        if (HMODE != 0) fwht32_stages_2_to_16(P);

        float v[32];
#pragma unroll
        for (int i = 0; i < 16; ++i) unpack2(P[i], v[2 * i], v[2 * i + 1]);
        float amax = max3_abs(v[0], v[1], v[2]);
#pragma unroll
        for (int j = 3; j < 31; j += 2) amax = max3_abs(amax, v[j], v[j + 1]);
        amax = fmaxf(amax, fabsf(v[31]));
        const uint32_t E = __float_as_uint(amax) >> 23;
        const uint32_t byte = E > 2u ? E - 2u : 0u;   // E <= 255 keeps byte <= 253 < 255
        const float mult = __uint_as_float((254u - byte) << 23);
        const uint64_t mult2 = pack2(mult, mult);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint64_t sp = mul2(P[i], mult2);
            unpack2(sp, v[2 * i], v[2 * i + 1]);       // v now holds the scaled values
        }

        uint32_t packed[4];
        if (SR == 0) {
#pragma unroll
            for (int q = 0; q < 4; ++q)
                packed[q] = cvt_e2m1x8(v[8 * q], v[8 * q + 1], v[8 * q + 2], v[8 * q + 3], v[8 * q + 4],
                                       v[8 * q + 5], v[8 * q + 6], v[8 * q + 7]);
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
                        w |= sr_e2m1(v[j], u8) << (4 * i);
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
