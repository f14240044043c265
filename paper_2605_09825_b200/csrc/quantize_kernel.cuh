// MXFP4 quantize kernel (Appendix A.1 Eq. (1), rotation of Appendix A.2, block orientation of
// Appendix D), one persistent CTA per SM.
//
// Work unit: a tile of 128 operand rows x 128 elements along K (4 MX blocks).  A producer warp
// streams source tiles into a ring of shared-memory stages with TMA.  The 512 consumer threads
// form groups (four of 128 threads, see QuantShape) that take alternate tiles; a thread handles
// 32-element blocks of its group's tile two at a time, each entirely in registers, so the five
// butterfly stages (as packed fp32x2 operations), the block maximum and the rounding need no
// cross-lane traffic.  The groups synchronise only among themselves, so they sit in different
// phases (one in its integer/convert instructions while another is in its floating-point ones)
// instead of all sixteen warps queueing on the same pipe at the same time.
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
    alignas(1024) uint8_t code_tile[4][kQCodeTileBytes];       // [consumer group * buffers + buffer]
    alignas(128) uint8_t scale_tile[4][kQScaleTileBytes];
    alignas(8) uint64_t full[kQStages];
    uint64_t empty[kQStages];
    int abort_flag;
};

// Sign diagonal of the randomized rotation as XOR words for raw bf16 data (all zero otherwise):
// pair[i] flips elements 2i (bit 15) and 2i+1 (bit 31) of a word holding two consecutive elements;
// word[k] = 0x80008000 if element k is flipped, for words holding element k of two columns (or
// one zero-extended element).  Built on the host from the 32-bit mask; read as constant-bank
// operands, so a flip costs one logic instruction per loaded word.
struct QuantSigns {
    uint32_t pair[16];
    uint32_t word[32];
};

struct QuantParams {
    QuantSigns signs;
    uint8_t* scales;
    int64_t outer, K;        // operand view
    int64_t nt;              // K / 32
    int32_t tiles_o, tiles_k;
    PhiloxRoundKeys rk;      // round keys of the stochastic-rounding stream (from the seed)
    uint32_t tag, sign_mask;
    int32_t scale_layout;    // 0 canonical, 1 tiled
    int32_t block2d;         // 0: 1 x 32 blocks, 1: 32 x 32 blocks (scale shared by 32 operand rows)
};

// One tensor to quantize: its source and code tensor maps plus parameters.  A launch takes two
// jobs (the second may be empty) so that both operands of a linear pass go through one kernel:
// the tail of the first tensor overlaps the start of the second and one launch gap disappears.
struct QuantJob {
    CUtensorMap tm_src;
    CUtensorMap tm_codes;
    QuantParams p;
    int32_t tiles;           // tiles_o * tiles_k, 0 for an empty job
};
// Both jobs as one kernel parameter: indexing it with the (block-uniform) job number reads the
// fields straight from parameter space instead of holding both sets in registers.
struct QuantJobs {
    QuantJob j[2];
};

// Packed fp32 pairs: sm_100 adds, multiplies and fuses two independent fp32 values held in a
// float2 (an aligned register pair) with a single instruction; each lane is an ordinary IEEE
// fp32 round-to-nearest operation, so results are bit-identical to the scalar form.  a - b is
// formed as fma(b, -1, a): the product is exact, so there is still exactly one rounding.
__device__ __forceinline__ float2 sub2(float2 a, float2 b)
{
    return __ffma2_rn(b, make_float2(-1.0f, -1.0f), a);
}

// max(|a|, |b|, |c|) in one instruction.
__device__ __forceinline__ float max3_abs(float a, float b, float c)
{
    float r;
    asm("max.abs.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// HMODE: 0 none | 1 deterministic H32 | 2 randomized H32 | 3 deterministic H16 | 4 randomized
// H16 (two independent 16-point transforms per MX block = the 32-point butterfly without its
// last stage; the randomized form repeats the low 16 sign bits for the second half).
//
// In-register 32-point Walsh-Hadamard transform of v[0..31] held as 16 pairs
// P[i] = (v[2i], v[2i+1]).  Stage h = 1 is applied while the pairs are formed (its partners
// share a pair); stages h = 2, 4, 8, 16 pair whole registers, so each packed add/sub does two
// butterflies.  Same five stages, same order, one fp32 rounding per output.
template <int HP>
__device__ __forceinline__ void fwht32_pair_stage(float2 (&P)[16])
{
#pragma unroll
    for (int i = 0; i < 16; i += 2 * HP) {
#pragma unroll
        for (int j = i; j < i + HP; ++j) {
            const float2 a = P[j], b = P[j + HP];
            P[j] = __fadd2_rn(a, b);
            P[j + HP] = sub2(a, b);
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

// Stochastic rounding (8 random bits per element, round up iff (u8 + 1/2) / 256 < frac) of two
// scaled values at a time.  |s| * 2^-126 re-biases a value so that bits 22.. of its fp32 pattern
// are the E2M1 magnitude code below it and bits 0..21 the position x between the two neighbouring
// grid points (the product is rounded toward +inf, so nothing below the pattern's last bit is
// lost to the strict comparison).  The rule compares x with T = (2 u8 + 1) * 2^13, and
// x > T  <=>  ceil(x / 2^13) > 2 u8 + 1, so a 13-bit number y = ceil(pattern / 2^13) = code * 512 +
// position-in-512ths carries everything the decision needs: the rounded code is
// (y + 510 - 2 u8) >> 9.  Two such numbers fit the halves of one register: z = 8 * pattern +
// 0x01FEFFF8 has y + 510 in its upper half, one byte permute packs the upper halves of two z,
// one multiply-add subtracts twice the two random bytes (spread to the halves by another
// permute; no borrow crosses the halves because y + 510 >= 2 u8), and shift, mask and a
// two-way minimum with 7 (values in [6, 8) may step to 8) give both codes.  Returns the codes in
// bits 0..3 and 16..19, sign bits included; `rbytes` holds the two random bytes in its bytes 0 and 2.
__device__ __forceinline__ uint32_t sr_e2m1_pair(float sa, float sb, uint32_t rbytes)
{
    const uint32_t za = __float_as_uint(__fmul_ru(fabsf(sa), 1.1754943508222875e-38f)) * 8u + 0x01FEFFF8u;
    const uint32_t zb = __float_as_uint(__fmul_ru(fabsf(sb), 1.1754943508222875e-38f)) * 8u + 0x01FEFFF8u;
    const uint32_t y2 = prmt(za, zb, 0x7632u);                       // (y_b + 510) << 16 | (y_a + 510)
    const uint32_t r2 = rbytes * 0xFFFFFFFEu + y2;                    // minus 2 u8 in each half
    const uint32_t mag = min_u16x2((r2 >> 9) & 0x000F000Fu, 0x00070007u);
    // bytes 0 and 2 = the top bytes of sa and sb with their sign bit replicated (selector nibble 8 | index)
    const uint32_t sg = prmt(__float_as_uint(sa), __float_as_uint(sb), 0xFFBBu);
    return mag | (sg & 0x00080008u);
}

// h = 1 butterfly of the deterministic rotation straight from bf16: (a + b, a - b) with a the
// bf16 value in the low 16 bits of `a_bits` and b already widened to fp32.  The mixed-precision
// add/sub widen a exactly, so the result equals the fp32 operation on the widened value.
__device__ __forceinline__ float2 first_stage_pair_bf16(uint32_t a_bits, float b)
{
    float s, d;
    const unsigned short a16 = static_cast<unsigned short>(a_bits);
    asm("add.rn.f32.bf16 %0, %1, %2;" : "=f"(s) : "h"(a16), "f"(b));
    asm("sub.rn.f32.bf16 %0, %1, %2;" : "=f"(d) : "h"(a16), "f"(b));
    return make_float2(s, d);
}

// One 32-element block out of a shared-memory stage into registers as 16 pairs.  The sign
// diagonal of the randomized modes is applied to the raw bf16 bits (a sign flip commutes with the
// exact widening), after which every rotated mode takes the same mixed-precision first butterfly
// stage; without rotation the pair is just widened.
template <int AXIS, int HMODE>
__device__ __forceinline__ void load_block(const uint8_t* stage, int kb, int o, const QuantSigns& sg,
                                           float2 (&P)[16])
{
    constexpr bool kRand = HMODE == 2 || HMODE == 4;
    if (AXIS == 1) {
        const uint8_t* base = stage + (kb >> 1) * (kQStageBytes / 2) + o * 128;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int chunk = (((kb & 1) * 4 + j) ^ (o & 7)) * 16;
            const uint4 q = smem_load<uint4>(base + chunk, stage, kQStageBytes);
            const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t wv = kRand ? (w[i] ^ sg.pair[4 * j + i]) : w[i];
                P[4 * j + i] = HMODE != 0 ? first_stage_pair_bf16(wv, __uint_as_float(wv & 0xFFFF0000u))
                                          : make_float2(__uint_as_float(wv << 16), __uint_as_float(wv & 0xFFFF0000u));
            }
        }
    } else {
        const uint16_t* base = reinterpret_cast<const uint16_t*>(stage) + (kb * 32) * 128 + o;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            // zero-extended elements; the flip word's upper half falls off in the shift / the 16-bit operand
            uint32_t a = smem_load<uint16_t>(base + (2 * i) * 128, stage, kQStageBytes);
            uint32_t b = smem_load<uint16_t>(base + (2 * i + 1) * 128, stage, kQStageBytes);
            if (kRand) {
                a ^= sg.word[2 * i];
                b ^= sg.word[2 * i + 1];
            }
            P[i] = HMODE != 0 ? first_stage_pair_bf16(a, __uint_as_float(b << 16))
                              : make_float2(__uint_as_float(a << 16), __uint_as_float(b << 16));
        }
    }
}

// Remaining butterfly stages and the block maximum.
template <int HMODE>
__device__ __forceinline__ float rotate_and_amax(float2 (&P)[16])
{
    if (HMODE != 0) {
        fwht32_pair_stage<1>(P);
        fwht32_pair_stage<2>(P);
        fwht32_pair_stage<4>(P);
        if (HMODE <= 2) fwht32_pair_stage<8>(P);   // the 16-point variant stops after h = 8
    }
    float amax = max3_abs(P[0].x, P[0].y, P[1].x);
#pragma unroll
    for (int i = 1; i < 15; ++i) amax = max3_abs(amax, P[i].y, P[i + 1].x);
    return fmaxf(amax, fabsf(P[15].y));
}

// Largest of a non-negative float over the lanes named by `mask` (bit patterns of non-negative
// floats order like unsigned integers).
__device__ __forceinline__ float lanes_max(uint32_t mask, float v)
{
    return __uint_as_float(__reduce_max_sync(mask, __float_as_uint(v)));
}

// Scale byte from the block maximum, scaling, rounding, packing: 16 bytes of packed codes and
// the E8M0 byte out.  e0 = index of the block's first element in the operand view.
template <int SR>
__device__ __forceinline__ void scale_round_pack(const float2 (&P)[16], float amax, uint64_t e0,
                                                 const QuantParams& p, uint32_t (&packed)[4], uint32_t& byte)
{
    const uint32_t E = __float_as_uint(amax) >> 23;
    byte = E > 2u ? E - 2u : 0u;                  // E <= 255 keeps byte <= 253 < 255
    const float mult = __uint_as_float((254u - byte) << 23);
    const float2 mult2 = make_float2(mult, mult);
    float v[32];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float2 sp = __fmul2_rn(P[i], mult2);
        v[2 * i] = sp.x;
        v[2 * i + 1] = sp.y;
    }
    if (SR == 0) {
#pragma unroll
        for (int q = 0; q < 4; ++q)
            packed[q] = cvt_e2m1x8(v[8 * q], v[8 * q + 1], v[8 * q + 2], v[8 * q + 3], v[8 * q + 4],
                                   v[8 * q + 5], v[8 * q + 6], v[8 * q + 7]);
    } else {
        const uint64_t g = e0 >> 4;                 // two 16-element Philox groups per block
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            uint32_t r[4];
            const uint64_t gg = g + half;
            philox4x32_10(static_cast<uint32_t>(gg), static_cast<uint32_t>(gg >> 32), p.tag, 0u, p.rk, r);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                // eight elements = four pairs -> one word of packed codes; element e of the 16-group
                // draws byte (e & 3) of word (e >> 2): pair j of this word uses bytes 0, 1 or 2, 3 of
                // word 2q + j / 2
                uint32_t c2[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int e = q * 8 + 2 * j;             // even element of the pair in the 16-group
                    const uint32_t rb = prmt(r[e >> 2], 0u, (j & 1) ? 0x4342u : 0x4140u);   // [u8_a, 0, u8_b, 0]
                    c2[j] = sr_e2m1_pair(v[half * 16 + e], v[half * 16 + e + 1], rb);
                }
                // bytes: codes of the even elements in the lower halves, of the odd ones in the upper
                const uint32_t u01 = c2[1] * 256u + c2[0], u23 = c2[3] * 256u + c2[2];
                const uint32_t even4 = prmt(u01, u23, 0x5410u), odd4 = prmt(u01, u23, 0x7632u);
                packed[half * 2 + q] = odd4 * 16u + even4;   // element k even in the low nibble
            }
        }
    }
}

// One block owned by one thread, whose warp holds 32 consecutive operand rows of the same block
// column: with 32 x 32 blocks (Appendix D) the maximum is taken over the warp.
template <int HMODE, int SR, bool PLAIN = false>
__device__ __forceinline__ void quantize_block(float2 (&P)[16], uint64_t e0, const QuantParams& p,
                                               uint32_t (&packed)[4], uint32_t& byte)
{
    float amax = rotate_and_amax<HMODE>(P);
    if (!PLAIN && p.block2d) amax = lanes_max(0xFFFFFFFFu, amax);
    scale_round_pack<SR>(P, amax, e0, p, packed, byte);
}

// tile index of a job -> (operand-row tile, K tile); the fastest-varying index walks the source's
// contiguous axis
template <int AXIS>
__device__ __forceinline__ void tile_coords(const QuantParams& p, int tile, int& to, int& tk)
{
    if (AXIS == 1) { to = tile / p.tiles_k; tk = tile % p.tiles_k; }
    else           { tk = tile / p.tiles_o; to = tile % p.tiles_o; }
}

template <int AXIS>
__device__ __forceinline__ void issue_tile_load(const CUtensorMap* tm_src, const QuantParams& p, int tile,
                                                uint8_t* stage, uint64_t* full)
{
    int to, tk;
    tile_coords<AXIS>(p, tile, to, tk);
    mbar_arrive_expect_tx(full, kQStageBytes);
    if (AXIS == 1) {
        tma_load_2d(stage, tm_src, full, tk * kQTileK, to * kQTileO);
        tma_load_2d(stage + kQStageBytes / 2, tm_src, full, tk * kQTileK + 64, to * kQTileO);
    } else {
        tma_load_2d(stage, tm_src, full, to * kQTileO, tk * kQTileK);
    }
}

// Consumer groups: four groups of 128 threads, each thread doing a tile's blocks in two sub-passes
// with a single staging buffer per group.  Each scheduler then holds one warp of every group --
// four different phases instead of the two that two groups of 256 threads give -- which keeps the
// FMA and ALU pipes busier: 5-10 % faster for the rotations and for stochastic rounding, no
// change for the un-rotated variant.
template <int HMODE, int SR>
struct QuantShape {
    static constexpr int kGroupThreads = 128;
    static constexpr int kGroups = kQConsumers / kGroupThreads;
    static constexpr int kSub = 256 / kGroupThreads;
    static constexpr int kBufs = kGroups == 2 ? 2 : 1;
};

// One tile of one job, as seen by a consumer thread: wait for the stage, rotate + quantize this
// thread's blocks (two at a time, two sub-passes), stage codes and scales, and (thread 0 of the
// group) store them.  `p` and `tm_codes` refer to kernel parameters, so every field is a
// constant-bank operand.  Returns false when a wait gave up (the group leaves the kernel).
// PLAIN: the tiled scale layout and 1 x 32 blocks are known at compile time (what the fused passes
// use); otherwise both are read from the parameters.
template <int AXIS, int HMODE, int SR, bool PLAIN>
__device__ __forceinline__ bool consume_tile(QuantSmem& sm, const QuantParams& p, const CUtensorMap* tm_codes,
                                             int tile, int it, int trip, int grp, int t)
{
    using Shape = QuantShape<HMODE, SR>;
    const int s = it % kQStages;
    const uint32_t round = it / kQStages;
    const int slot = grp * Shape::kBufs + (Shape::kBufs == 2 ? (trip & 1) : 0);   // staging tile of this trip
    int to, tk;
    tile_coords<AXIS>(p, tile, to, tk);

    const bool ok = mbar_wait(&sm.full[s], round & 1, &sm.abort_flag);
    if (Shape::kBufs == 1) {
        // single staging buffer: last trip's store must have read it before anyone rewrites it
        if (t == 0) bulk_wait_group_read<0>();
        asm volatile("barrier.cta.sync %0, %1;" ::"r"(grp + 1), "n"(Shape::kGroupThreads) : "memory");
    }

#pragma unroll
    for (int u = 0; u < Shape::kSub; ++u) {
        const int tv = t + u * Shape::kGroupThreads;   // position in the 256-thread layout of a tile
        const int kbh = tv >> 7;                       // this thread's blocks along K: kbh and kbh + 2
        const int o = tv & 127;                        // operand row inside the tile
        float2 P0[16], P1[16];
        // (after a failed wait the stage holds whatever it held: the blocks are still worked
        // through, nothing computed from them leaves the CTA)
        load_block<AXIS, HMODE>(&sm.stage[s][0], kbh, o, p.signs, P0);
        load_block<AXIS, HMODE>(&sm.stage[s][0], kbh + 2, o, p.signs, P1);
        if (u == Shape::kSub - 1) {
            // the stage is in registers now: hand it back to the producer
            __syncwarp();
            if ((t & 31) == 0) mbar_arrive(&sm.empty[s]);
        }

        const uint64_t e_row = static_cast<uint64_t>(to * kQTileO + o) * static_cast<uint64_t>(p.K);
        uint32_t packed0[4], packed1[4], byte0, byte1;
        quantize_block<HMODE, SR, PLAIN>(P0, e_row + static_cast<uint64_t>((tk * 4 + kbh) * 32), p, packed0, byte0);
        quantize_block<HMODE, SR, PLAIN>(P1, e_row + static_cast<uint64_t>((tk * 4 + kbh + 2) * 32), p, packed1, byte1);

        // stage the results: codes in the 64-byte swizzle the TMA store expects
        uint8_t* ct = &sm.code_tile[slot][o * 64];
        smem_store(ct + ((kbh ^ ((o >> 1) & 3)) * 16), make_uint4(packed0[0], packed0[1], packed0[2], packed0[3]),
                   sm.code_tile[slot], kQCodeTileBytes);
        smem_store(ct + (((kbh + 2) ^ ((o >> 1) & 3)) * 16), make_uint4(packed1[0], packed1[1], packed1[2], packed1[3]),
                   sm.code_tile[slot], kQCodeTileBytes);
        if (PLAIN || p.scale_layout == 1) {
            uint8_t* st = &sm.scale_tile[slot][(o & 31) * 16 + (o >> 5) * 4];
            smem_store(st + kbh, static_cast<uint8_t>(byte0), sm.scale_tile[slot], kQScaleTileBytes);
            smem_store(st + kbh + 2, static_cast<uint8_t>(byte1), sm.scale_tile[slot], kQScaleTileBytes);
        } else if (ok) {
            const int64_t og = static_cast<int64_t>(to) * kQTileO + o;
            const int64_t tg = static_cast<int64_t>(tk) * 4 + kbh;
            if (og < p.outer && tg < p.nt) p.scales[og * p.nt + tg] = static_cast<uint8_t>(byte0);
            if (og < p.outer && tg + 2 < p.nt) p.scales[og * p.nt + tg + 2] = static_cast<uint8_t>(byte1);
        }
    }
    fence_proxy_async_smem();
    // double-buffered staging: the store this group issued one trip ago must have drained its
    // buffer before the next trip (which every thread of the group reaches only through the
    // barrier below) overwrites it
    if (Shape::kBufs == 2 && t == 0) bulk_wait_group_read<0>();
    uint32_t any_fail;
    asm volatile(
        "{\n\t.reg .pred P, Q;\n\t"
        "setp.ne.u32 Q, %1, 0;\n\t"
        "barrier.cta.red.or.pred P, %2, %3, Q;\n\t"
        "selp.u32 %0, 1, 0, P;\n\t}"
        : "=r"(any_fail)
        : "r"(ok ? 0u : 1u), "r"(grp + 1), "n"(Shape::kGroupThreads)
        : "memory");
    if (any_fail) return false;
    if (t == 0) {
        tma_store_2d(tm_codes, &sm.code_tile[slot][0], tk * (kQTileK / 2), to * kQTileO);
        if (PLAIN || p.scale_layout == 1)
            bulk_store_1d(p.scales + (static_cast<int64_t>(to) * p.tiles_k + tk) * kQScaleTileBytes,
                          &sm.scale_tile[slot][0], kQScaleTileBytes);
        bulk_commit_group();
    }
    return true;
}

template <int AXIS0, int AXIS1, int HMODE, int SR, bool PLAIN>
__global__ void __launch_bounds__(kQThreads, 1)
quantize_kernel(const __grid_constant__ QuantJobs jobs)
{
    using Shape = QuantShape<HMODE, SR>;
    extern __shared__ uint8_t smem_raw[];
    // ld.shared / st.shared (address space kept visible) for the un-rotated round-to-nearest variant,
    // 8 % faster row-wise that way; the others sit at the 96-register limit, where the extra live
    // shared addresses turn into spills (row-wise stochastic rounding 84 -> 95 us on 8192 x 14336,
    // rotated round-to-nearest 2-4 % slower, column-wise equal), and keep generic accesses.
    QuantSmem& sm = *reinterpret_cast<QuantSmem*>(
        (HMODE == 0 && SR == 0) ? smem_align_1024(smem_raw) : smem_align_1024_generic(smem_raw));
    const int tid = threadIdx.x;
    const int tiles0 = jobs.j[0].tiles;
    const int total_tiles = tiles0 + jobs.j[1].tiles;
    const int my_tiles = blockIdx.x < total_tiles ? (total_tiles - 1 - blockIdx.x) / gridDim.x + 1 : 0;

    if (tid == 0) {
        sm.abort_flag = 0;
        for (int s = 0; s < kQStages; ++s) {
            mbar_init(&sm.full[s], 1);
            mbar_init(&sm.empty[s], Shape::kGroupThreads / 32);   // the warps of one consumer group
        }
        fence_barrier_init();
    }
    __syncthreads();
    griddep_launch_dependents();
    griddep_wait();        // no global-memory access before the previous kernel in the stream is done

    if (tid >= kQConsumers) {
        // ------------------------------------------------------------ producer warp
        if (tid == kQConsumers) {
            tma_prefetch_desc(&jobs.j[0].tm_src);
            if (jobs.j[1].tiles > 0) tma_prefetch_desc(&jobs.j[1].tm_src);
            for (int it = 0; it < my_tiles; ++it) {
                const int tile = blockIdx.x + it * gridDim.x;
                const int s = it % kQStages;
                const uint32_t round = it / kQStages;
                if (round > 0 && !mbar_wait(&sm.empty[s], (round - 1) & 1, &sm.abort_flag)) break;
                if (tile < tiles0)
                    issue_tile_load<AXIS0>(&jobs.j[0].tm_src, jobs.j[0].p, tile, &sm.stage[s][0], &sm.full[s]);
                else
                    issue_tile_load<AXIS1>(&jobs.j[1].tm_src, jobs.j[1].p, tile - tiles0, &sm.stage[s][0],
                                           &sm.full[s]);
            }
        }
        return;
    }

    // ---------------------------------------------------------------- consumers
    const int grp = tid / Shape::kGroupThreads;     // consumer group: takes tiles grp, grp + kGroups, ...
    const int t = tid % Shape::kGroupThreads;
    if (t == 0) {
        tma_prefetch_desc(&jobs.j[0].tm_codes);
        if (jobs.j[1].tiles > 0) tma_prefetch_desc(&jobs.j[1].tm_codes);
    }

    // this CTA's tiles come in increasing order: first those of job 0, then those of job 1, each
    // through a loop specialised for that job's axis and parameters
    int it = grp, trip = 0;
    bool alive = true;
    for (; it < my_tiles; it += Shape::kGroups, ++trip) {
        const int gtile = blockIdx.x + it * gridDim.x;
        if (gtile >= tiles0) break;
        alive = consume_tile<AXIS0, HMODE, SR, PLAIN>(sm, jobs.j[0].p, &jobs.j[0].tm_codes, gtile, it, trip, grp, t);
        if (!alive) break;
    }
    if (alive) {
        for (; it < my_tiles; it += Shape::kGroups, ++trip) {
            const int gtile = blockIdx.x + it * gridDim.x;
            if (!consume_tile<AXIS1, HMODE, SR, PLAIN>(sm, jobs.j[1].p, &jobs.j[1].tm_codes, gtile - tiles0, it, trip,
                                                grp, t))
                break;
        }
    }
    if (t == 0) bulk_wait_group<0>();
}

}  // namespace mxfp4
