// One-read dual-axis MXFP4 quantize: the row-wise operand (blocks along the contiguous axis)
// AND the column-wise, transposed operand (blocks down the rows; Appendix D's two 1D
// orientations, or its 32 x 32 strategy for both) of one bf16 tensor from a single pass over
// it.  A linear layer needs every one of X, W and dY in both orientations (Appendix C: Fprop
// and Wgrad for X, Fprop and Dgrad for W, Dgrad and Wgrad for dY), so this replaces two reads
// of 2 bytes per element by one: 3.06 instead of 5.06 bytes of traffic per element.
//
// Same skeleton as the single-axis kernel: persistent CTAs, a TMA producer warp filling a ring
// of 128 x 128 source tiles (two 128-row x 64-column boxes in the 128-byte swizzle), consumer
// groups on alternate tiles (two of 256 threads or four of 128, see QuantDualShape).  Per tile
// and sub-pass a thread first handles two row-wise blocks (its source row, block columns kbh and
// kbh + 2), then two column-wise blocks:
// it reads 32 rows of one 4-byte word, i.e. of two adjacent source columns, which gives it the
// same block of two neighbouring operand rows of the transposed operand.  Each orientation has
// its own staged code / scale tile and its own TMA store.
#pragma once

#include "quantize_kernel.cuh"

namespace mxfp4 {

constexpr int kQDStages = 4;
// Consumer-group width per variant.  256: two groups of 256 threads on alternate tiles, double-
// buffered staging.  128: four groups of 128 threads, each thread doing a tile's blocks in two
// sub-passes, single-buffered staging -- four different phases per scheduler instead of two, which
// keeps the FMA and ALU pipes busier for the deterministic rotations (7-9 % faster there) but
// costs the un-rotated variant and the stochastic-rounding ones 5-20 % here (the kernel has
// less register headroom than the single-axis one) and changes nothing for the randomized rotations.
template <int HMODE, int SR>
struct QuantDualShape {
    static constexpr int kGroupThreads = (HMODE != 0 && SR == 0) ? 128 : 256;
    static constexpr int kGroups = kQConsumers / kGroupThreads;
    static constexpr int kSub = 256 / kGroupThreads;
    static constexpr int kBufs = kGroups == 2 ? 2 : 1;
    // The un-rotated round-to-nearest variant does so little arithmetic that it runs at the HBM
    // bound (16384 x 14336 in 111-117 us back to back = 0.99 of the copy bandwidth) -- in the
    // kernel's first form.  Each of the later savings makes THAT variant slower, measured one by
    // one on one GPU: ld.shared / st.shared instead of generic accesses 139 us, the compile-time
    // layout (PLAIN) 138, the L2 prefetch of the next tile 152; every other variant gains from
    // each of them (deterministic H32 150 -> 134 us, stochastic rounding 342 -> 288).  Consumers
    // that run ahead seem to bunch the memory requests of a kernel that has no arithmetic to
    // hide them behind; the variant therefore keeps the first form.
    static constexpr bool kFirstForm = HMODE == 0 && SR == 0;
};

struct QuantDualSmem {
    alignas(1024) uint8_t stage[kQDStages][kQStageBytes];
    alignas(1024) uint8_t code_tile[8][kQCodeTileBytes];     // [(group * buffers + buffer) * 2 + orientation]
    alignas(128) uint8_t scale_tile[8][kQScaleTileBytes];
    alignas(8) uint64_t full[kQDStages];
    uint64_t empty[kQDStages];
    int abort_flag;
};

struct QuantDualJob {
    CUtensorMap tm_src;          // [rows x cols] bf16, box 128 x 64, 128-byte swizzle
    CUtensorMap tm_codes_row;    // row-wise operand codes   [rows x cols/2]
    CUtensorMap tm_codes_col;    // column-wise operand codes [cols x rows/2]
    QuantParams pr;              // row-wise operand:    outer = rows, K = cols
    QuantParams pc;              // column-wise operand: outer = cols, K = rows
    int32_t tiles_r, tiles_c;    // source tiles of 128 rows / 128 columns
};

// Two column-wise blocks out of the swizzled stage: rows kb*32 .. kb*32+31 of source columns
// 2*jc (-> PA) and 2*jc + 1 (-> PB), as 16 pairs each, sign diagonal and first butterfly stage
// applied on the way in.  Element (r, c) of the tile sits at
//   (c / 64) * 16384 + r * 128 + (((c % 64) / 8) ^ (r % 8)) * 16 + (c % 8) * 2.
template <int HMODE>
__device__ __forceinline__ void load_column_blocks(const uint8_t* stage, int kb, int jc, const QuantSigns& sg,
                                                   float2 (&PA)[16], float2 (&PB)[16])
{
    const int w = jc & 31;                                  // 4-byte word inside the 128-byte row
    const uint32_t base = (jc >> 5) * (kQStageBytes / 2) + kb * (32 * 128) + ((w >> 2) << 4) + (w & 3) * 4;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const int r0 = 2 * i, r1 = 2 * i + 1;               // rows of the block; (kb*32 + r) % 8 == r % 8
        uint32_t w0 = smem_load<uint32_t>(stage + ((base ^ ((r0 & 7) << 4)) + r0 * 128), stage, kQStageBytes);
        uint32_t w1 = smem_load<uint32_t>(stage + ((base ^ ((r1 & 7) << 4)) + r1 * 128), stage, kQStageBytes);
        if (HMODE == 2 || HMODE == 4) {                     // element r of both columns shares its sign
            w0 ^= sg.word[r0];
            w1 ^= sg.word[r1];
        }
        if (HMODE != 0) {
            PA[i] = first_stage_pair_bf16(w0, __uint_as_float(w1 << 16));
            PB[i] = first_stage_pair_bf16(w0 >> 16, __uint_as_float(w1 & 0xFFFF0000u));
        } else {
            PA[i] = make_float2(__uint_as_float(w0 << 16), __uint_as_float(w1 << 16));
            PB[i] = make_float2(__uint_as_float(w0 & 0xFFFF0000u), __uint_as_float(w1 & 0xFFFF0000u));
        }
    }
}

// Stage one block's results: codes into the 64-byte-swizzled code tile, the scale byte into the
// 512-byte scale tile (tiled layout) or straight to global memory (canonical layout).
template <bool TILED = false>
__device__ __forceinline__ void stage_block(uint8_t* code_tile, uint8_t* scale_tile, const QuantParams& p, int o,
                                            int kb, int to, int tk, const uint32_t (&packed)[4], uint32_t byte,
                                            bool ok)
{
    smem_store(code_tile + o * 64 + ((kb ^ ((o >> 1) & 3)) * 16), make_uint4(packed[0], packed[1], packed[2], packed[3]),
               code_tile, kQCodeTileBytes);
    if (TILED || p.scale_layout == 1) {
        smem_store(scale_tile + (o & 31) * 16 + (o >> 5) * 4 + kb, static_cast<uint8_t>(byte), scale_tile,
                   kQScaleTileBytes);
    } else if (ok) {
        const int64_t og = static_cast<int64_t>(to) * kQTileO + o;
        const int64_t tg = static_cast<int64_t>(tk) * 4 + kb;
        if (og < p.outer && tg < p.nt) p.scales[og * p.nt + tg] = static_cast<uint8_t>(byte);
    }
}

// PLAIN: the tiled scale layout and 1 x 32 blocks are known at compile time (the layer-level path);
// otherwise both are read from the job.
template <int HMODE, int SR, bool PLAIN>
__global__ void __launch_bounds__(kQThreads, 1)
quantize_dual_kernel(const __grid_constant__ QuantDualJob job)
{
    using Shape = QuantDualShape<HMODE, SR>;
    constexpr int kQDGroupThreads = Shape::kGroupThreads, kQDGroups = Shape::kGroups, kQDSub = Shape::kSub,
                  kQDBufs = Shape::kBufs;
    extern __shared__ uint8_t smem_raw[];
    QuantDualSmem& sm = *reinterpret_cast<QuantDualSmem*>(
        Shape::kFirstForm ? smem_align_1024_generic(smem_raw) : smem_align_1024(smem_raw));
    const int tid = threadIdx.x;
    const int total_tiles = job.tiles_r * job.tiles_c;
    const int my_tiles = blockIdx.x < total_tiles ? (total_tiles - 1 - blockIdx.x) / gridDim.x + 1 : 0;

    if (tid == 0) {
        sm.abort_flag = 0;
        for (int s = 0; s < kQDStages; ++s) {
            mbar_init(&sm.full[s], 1);
            mbar_init(&sm.empty[s], kQDGroupThreads / 32);  // the warps of one consumer group
        }
        fence_barrier_init();
    }
    __syncthreads();
    griddep_launch_dependents();
    griddep_wait();        // no global-memory access before the previous kernel in the stream is done

    if (tid >= kQConsumers) {
        // ------------------------------------------------------------ producer warp
        if (tid == kQConsumers) {
            tma_prefetch_desc(&job.tm_src);
            for (int it = 0; it < my_tiles; ++it) {
                const int tile = blockIdx.x + it * gridDim.x;
                const int tr = tile / job.tiles_c, tc = tile % job.tiles_c;   // walk the contiguous axis first
                const int s = it % kQDStages;
                const uint32_t round = it / kQDStages;
                if (round > 0 && !mbar_wait(&sm.empty[s], (round - 1) & 1, &sm.abort_flag)) break;
                mbar_arrive_expect_tx(&sm.full[s], kQStageBytes);
                tma_load_2d(&sm.stage[s][0], &job.tm_src, &sm.full[s], tc * 128, tr * 128);
                tma_load_2d(&sm.stage[s][kQStageBytes / 2], &job.tm_src, &sm.full[s], tc * 128 + 64, tr * 128);
                // the tile this stage takes next goes to L2 now: its load is issued only when the
                // stage comes back, three quarters into the tile after this one of its group, and
                // would otherwise wait for HBM with a quarter of a tile's time to hide it in
                if (!Shape::kFirstForm && it + kQDStages < my_tiles) {
                    const int nt = tile + kQDStages * gridDim.x;
                    const int ntr = nt / job.tiles_c, ntc = nt % job.tiles_c;
                    tma_prefetch_l2_2d(&job.tm_src, ntc * 128, ntr * 128);
                    tma_prefetch_l2_2d(&job.tm_src, ntc * 128 + 64, ntr * 128);
                }
            }
        }
        return;
    }

    // ---------------------------------------------------------------- consumers
    const int grp = tid / kQDGroupThreads;     // consumer group: takes tiles grp, grp + kQDGroups, ...
    const int t = tid % kQDGroupThreads;
    // the 16 lanes that share a 32-column group (a 32 x 32 region of the transposed operand)
    const uint32_t half_mask = (tid & 16) ? 0xFFFF0000u : 0x0000FFFFu;
    const QuantParams& pr = job.pr;
    const QuantParams& pc = job.pc;
    if (t == 0) {
        tma_prefetch_desc(&job.tm_codes_row);
        tma_prefetch_desc(&job.tm_codes_col);
    }

    int trip = 0;
    for (int it = grp; it < my_tiles; it += kQDGroups, ++trip) {
        const int tile = blockIdx.x + it * gridDim.x;
        const int tr = tile / job.tiles_c, tc = tile % job.tiles_c;
        const int s = it % kQDStages;
        const uint32_t round = it / kQDStages;
        const int slot = (grp * kQDBufs + (kQDBufs == 2 ? (trip & 1) : 0)) * 2;   // staging tiles of this trip
        const bool ok = mbar_wait(&sm.full[s], round & 1, &sm.abort_flag);
        if (kQDBufs == 1) {
            // single staging buffer: last trip's stores must have read it before anyone rewrites it
            if (t == 0) bulk_wait_group_read<0>();
            asm volatile("barrier.cta.sync %0, %1;" ::"r"(grp + 1), "n"(kQDGroupThreads) : "memory");
        }

        float2 P0[16], P1[16];
        uint32_t packed[4], byte;
#pragma unroll
        for (int u = 0; u < kQDSub; ++u) {
            const int tv = t + u * kQDGroupThreads;     // position in the 256-thread layout of a tile
            const int kbh = tv >> 7;                    // row-wise: blocks kbh and kbh + 2 of source row o
            const int o = tv & 127;
            const int kbc = tv >> 6;                    // column-wise: block kbc of source columns 2*jc, 2*jc + 1
            const int jc = tv & 63;

            // ---- row-wise operand: operand row = source row, K = columns
            // (after a failed wait the stage holds whatever it held: the blocks are still worked
            // through, nothing computed from them leaves the CTA; the first form zero-fills instead)
            if (!Shape::kFirstForm || ok) {
                load_block<1, HMODE>(&sm.stage[s][0], kbh, o, pr.signs, P0);
                load_block<1, HMODE>(&sm.stage[s][0], kbh + 2, o, pr.signs, P1);
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) P0[i] = P1[i] = make_float2(0.0f, 0.0f);
            }
            {
                const uint64_t e_row = static_cast<uint64_t>(tr * 128 + o) * static_cast<uint64_t>(pr.K);
                uint8_t* ct = &sm.code_tile[slot][0];
                uint8_t* st = &sm.scale_tile[slot][0];
                quantize_block<HMODE, SR, PLAIN>(P0, e_row + static_cast<uint64_t>((tc * 4 + kbh) * 32), pr, packed, byte);
                stage_block<PLAIN>(ct, st, pr, o, kbh, tr, tc, packed, byte, ok);
                quantize_block<HMODE, SR, PLAIN>(P1, e_row + static_cast<uint64_t>((tc * 4 + kbh + 2) * 32), pr, packed, byte);
                stage_block<PLAIN>(ct, st, pr, o, kbh + 2, tr, tc, packed, byte, ok);
            }

            // ---- column-wise operand: operand row = source column, K = rows
            if (!Shape::kFirstForm || ok) {
                load_column_blocks<HMODE>(&sm.stage[s][0], kbc, jc, pc.signs, P0, P1);
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) P0[i] = P1[i] = make_float2(0.0f, 0.0f);
            }
            if (u == kQDSub - 1) {
                // the stage is in registers now: hand it back to the producer
                __syncwarp();
                if ((tid & 31) == 0) mbar_arrive(&sm.empty[s]);
            }
            {
                float amax0 = rotate_and_amax<HMODE>(P0);
                float amax1 = rotate_and_amax<HMODE>(P1);
                if (!PLAIN && pc.block2d) amax0 = amax1 = lanes_max(half_mask, fmaxf(amax0, amax1));
                const uint64_t e_blk = static_cast<uint64_t>((tr * 4 + kbc) * 32);
                const uint64_t e_row = static_cast<uint64_t>(tc * 128 + 2 * jc) * static_cast<uint64_t>(pc.K);
                uint8_t* ct = &sm.code_tile[slot + 1][0];
                uint8_t* st = &sm.scale_tile[slot + 1][0];
                scale_round_pack<SR>(P0, amax0, e_row + e_blk, pc, packed, byte);
                stage_block<PLAIN>(ct, st, pc, 2 * jc, kbc, tc, tr, packed, byte, ok);
                scale_round_pack<SR>(P1, amax1, e_row + static_cast<uint64_t>(pc.K) + e_blk, pc, packed, byte);
                stage_block<PLAIN>(ct, st, pc, 2 * jc + 1, kbc, tc, tr, packed, byte, ok);
            }
        }

        fence_proxy_async_smem();
        // double-buffered staging: the stores this group issued one trip ago must have drained
        // their buffers before the next trip (which every thread of the group reaches only
        // through the barrier below) overwrites them
        if (kQDBufs == 2 && t == 0) bulk_wait_group_read<0>();
        uint32_t any_fail;
        asm volatile(
            "{\n\t.reg .pred P, Q;\n\t"
            "setp.ne.u32 Q, %1, 0;\n\t"
            "barrier.cta.red.or.pred P, %2, %3, Q;\n\t"
            "selp.u32 %0, 1, 0, P;\n\t}"
            : "=r"(any_fail)
            : "r"(ok ? 0u : 1u), "r"(grp + 1), "n"(kQDGroupThreads)
            : "memory");
        if (any_fail) break;
        if (t == 0) {
            tma_store_2d(&job.tm_codes_row, &sm.code_tile[slot][0], tc * 64, tr * 128);
            tma_store_2d(&job.tm_codes_col, &sm.code_tile[slot + 1][0], tr * 64, tc * 128);
            if (PLAIN || pr.scale_layout == 1) {
                bulk_store_1d(pr.scales + (static_cast<int64_t>(tr) * pr.tiles_k + tc) * kQScaleTileBytes,
                              &sm.scale_tile[slot][0], kQScaleTileBytes);
                bulk_store_1d(pc.scales + (static_cast<int64_t>(tc) * pc.tiles_k + tr) * kQScaleTileBytes,
                              &sm.scale_tile[slot + 1][0], kQScaleTileBytes);
            }
            bulk_commit_group();
        }
    }
    if (t == 0) bulk_wait_group<0>();
}

}  // namespace mxfp4
