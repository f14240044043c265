// MXFP8 quantize kernel for the passes the precision ladder leaves in 8 bits (Table 1): E4M3
// elements, one E8M0 scale per 32 elements along the reduction axis (Eq. (1) of Appendix A.1 with
// the 8-bit element format: scale 2^(floor(log2 amax) - 8), round to nearest even, saturating
// at 448), row-wise or column-wise blocks (Appendix D), no rotation, no stochastic rounding.
//
// Same skeleton as the 4-bit kernel (persistent CTAs, TMA producer warp, two consumer groups on
// alternate 128 x 128 tiles, one or two tensors per launch); a tile's codes are 128 rows x 128
// bytes, staged in the 128-byte swizzle for one TMA store.  3.03125 bytes per element.
#pragma once

#include "quantize_kernel.cuh"

namespace mxfp4 {

constexpr int kQ8CodeTileBytes = 128 * 128;

struct QuantFp8Smem {
    alignas(1024) uint8_t stage[kQStages][kQStageBytes];
    alignas(1024) uint8_t code_tile[2][2][kQ8CodeTileBytes];   // [consumer group][double buffer]
    alignas(128) uint8_t scale_tile[2][2][kQScaleTileBytes];
    alignas(8) uint64_t full[kQStages];
    uint64_t empty[kQStages];
    int abort_flag;
};

// Four E4M3 codes (one 32-bit word) from four floats; v0 lands in bits 7:0.
__device__ __forceinline__ uint32_t cvt_e4m3x4(float v0, float v1, float v2, float v3)
{
    uint32_t r;
    asm("{\n\t.reg .b16 lo, hi;\n\t"
        "cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1;\n\t"
        "cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3;\n\t"
        "mov.b32 %0, {lo, hi};\n\t}"
        : "=r"(r)
        : "f"(v0), "f"(v1), "f"(v2), "f"(v3));
    return r;
}

// One block: maximum, scale byte, scaling, conversion.  32 code bytes out.
__device__ __forceinline__ void quantize_block_fp8(float2 (&P)[16], uint32_t (&packed)[8], uint32_t& byte)
{
    const float amax = rotate_and_amax<0>(P);
    const uint32_t E = __float_as_uint(amax) >> 23;
    byte = E > 8u ? E - 8u : 0u;
    const float mult = __uint_as_float((254u - byte) << 23);
    const float2 mult2 = make_float2(mult, mult);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const float2 a = __fmul2_rn(P[2 * q], mult2), b = __fmul2_rn(P[2 * q + 1], mult2);
        packed[q] = cvt_e4m3x4(a.x, a.y, b.x, b.y);
    }
}

template <int AXIS>
__device__ __forceinline__ bool consume_tile_fp8(QuantFp8Smem& sm, const QuantParams& p, const CUtensorMap* tm_codes,
                                                 int tile, int it, int trip, int grp, int t)
{
    const int kbh = t >> 7;            // this thread's blocks along K: kbh and kbh + 2
    const int o = t & 127;             // operand row inside the tile
    const int s = it % kQStages;
    const uint32_t round = it / kQStages;
    const int buf = trip & 1;
    int to, tk;
    tile_coords<AXIS>(p, tile, to, tk);

    const bool ok = mbar_wait(&sm.full[s], round & 1, &sm.abort_flag);
    float2 P0[16], P1[16];
    if (ok) {
        load_block<AXIS, 0>(&sm.stage[s][0], kbh, o, p.signs, P0);
        load_block<AXIS, 0>(&sm.stage[s][0], kbh + 2, o, p.signs, P1);
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) P0[i] = P1[i] = make_float2(0.0f, 0.0f);
    }
    __syncwarp();
    if ((t & 31) == 0) mbar_arrive(&sm.empty[s]);

    uint32_t packed0[8], packed1[8], byte0, byte1;
    quantize_block_fp8(P0, packed0, byte0);
    quantize_block_fp8(P1, packed1, byte1);

    // codes: row o of the tile is 128 bytes = 8 chunks of 16, chunk c stored at c ^ (o % 8)
    uint8_t* ct = &sm.code_tile[grp][buf][o * 128];
    const int sw = o & 7;
    const void* ctb = sm.code_tile[grp][buf];
    smem_store(ct + (((2 * kbh) ^ sw) * 16), make_uint4(packed0[0], packed0[1], packed0[2], packed0[3]), ctb, 128 * 128);
    smem_store(ct + (((2 * kbh + 1) ^ sw) * 16), make_uint4(packed0[4], packed0[5], packed0[6], packed0[7]), ctb, 128 * 128);
    smem_store(ct + (((2 * kbh + 4) ^ sw) * 16), make_uint4(packed1[0], packed1[1], packed1[2], packed1[3]), ctb, 128 * 128);
    smem_store(ct + (((2 * kbh + 5) ^ sw) * 16), make_uint4(packed1[4], packed1[5], packed1[6], packed1[7]), ctb, 128 * 128);
    if (p.scale_layout == 1) {
        uint8_t* st = &sm.scale_tile[grp][buf][(o & 31) * 16 + (o >> 5) * 4];
        smem_store(st + kbh, static_cast<uint8_t>(byte0), sm.scale_tile[grp][buf], kQScaleTileBytes);
        smem_store(st + kbh + 2, static_cast<uint8_t>(byte1), sm.scale_tile[grp][buf], kQScaleTileBytes);
    } else if (ok) {
        const int64_t og = static_cast<int64_t>(to) * kQTileO + o;
        const int64_t tg = static_cast<int64_t>(tk) * 4 + kbh;
        if (og < p.outer && tg < p.nt) p.scales[og * p.nt + tg] = static_cast<uint8_t>(byte0);
        if (og < p.outer && tg + 2 < p.nt) p.scales[og * p.nt + tg + 2] = static_cast<uint8_t>(byte1);
    }
    fence_proxy_async_smem();
    if (t == 0) bulk_wait_group_read<0>();     // last trip's stores have drained this group's buffers
    uint32_t any_fail;
    asm volatile(
        "{\n\t.reg .pred P, Q;\n\t"
        "setp.ne.u32 Q, %1, 0;\n\t"
        "barrier.cta.red.or.pred P, %2, %3, Q;\n\t"
        "selp.u32 %0, 1, 0, P;\n\t}"
        : "=r"(any_fail)
        : "r"(ok ? 0u : 1u), "r"(grp + 1), "n"(kQConsumers / 2)
        : "memory");
    if (any_fail) return false;
    if (t == 0) {
        tma_store_2d(tm_codes, &sm.code_tile[grp][buf][0], tk * kQTileK, to * kQTileO);
        if (p.scale_layout == 1)
            bulk_store_1d(p.scales + (static_cast<int64_t>(to) * p.tiles_k + tk) * kQScaleTileBytes,
                          &sm.scale_tile[grp][buf][0], kQScaleTileBytes);
        bulk_commit_group();
    }
    return true;
}

template <int AXIS0, int AXIS1>
__global__ void __launch_bounds__(kQThreads, 1)
quantize_fp8_kernel(const __grid_constant__ QuantJobs jobs)
{
    extern __shared__ uint8_t smem_raw[];
    QuantFp8Smem& sm = *reinterpret_cast<QuantFp8Smem*>(smem_align_1024(smem_raw));
    const int tid = threadIdx.x;
    const int tiles0 = jobs.j[0].tiles;
    const int total_tiles = tiles0 + jobs.j[1].tiles;
    const int my_tiles = blockIdx.x < total_tiles ? (total_tiles - 1 - blockIdx.x) / gridDim.x + 1 : 0;

    if (tid == 0) {
        sm.abort_flag = 0;
        for (int s = 0; s < kQStages; ++s) {
            mbar_init(&sm.full[s], 1);
            mbar_init(&sm.empty[s], kQConsumers / 64);
        }
        fence_barrier_init();
    }
    __syncthreads();
    griddep_launch_dependents();
    griddep_wait();        // no global-memory access before the previous kernel in the stream is done

    if (tid >= kQConsumers) {
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

    const int grp = tid >> 8;
    const int t = tid & 255;
    if (t == 0) {
        tma_prefetch_desc(&jobs.j[0].tm_codes);
        if (jobs.j[1].tiles > 0) tma_prefetch_desc(&jobs.j[1].tm_codes);
    }
    int it = grp, trip = 0;
    bool alive = true;
    for (; it < my_tiles; it += 2, ++trip) {
        const int gtile = blockIdx.x + it * gridDim.x;
        if (gtile >= tiles0) break;
        alive = consume_tile_fp8<AXIS0>(sm, jobs.j[0].p, &jobs.j[0].tm_codes, gtile, it, trip, grp, t);
        if (!alive) break;
    }
    if (alive) {
        for (; it < my_tiles; it += 2, ++trip) {
            const int gtile = blockIdx.x + it * gridDim.x;
            if (!consume_tile_fp8<AXIS1>(sm, jobs.j[1].p, &jobs.j[1].tm_codes, gtile - tiles0, it, trip, grp, t))
                break;
        }
    }
    if (t == 0) bulk_wait_group<0>();
}

}  // namespace mxfp4
