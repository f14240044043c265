// Block-scaled MXFP4 GEMM on the 5th-generation tensor cores (the MXFP4 GEMM that replaces the
// linear layers' FP8 GEMM; operand orientation per Appendix C):
//
//   out[m][n] = alpha * sum_t 2^(sa[m][t]-127) 2^(sb[n][t]-127) sum_{k in block t} A[m][k] B[n][k]
//
// CTA-pair kernel (tcgen05 cta_group::2): the two CTAs of a cluster share one 256 x 384 output
// tile (two 256 x 192 MMAs per K = 64).  Each CTA loads its own 128 rows of A and its own
// 2 x 96 rows of B: 40 KB per K-step of 256 elements for 128 x 384 outputs, against the 48 KB a
// lone 128 x 256 tile needs for two thirds of that -- on operands that toggle, an FP4 GEMM here
// runs at the device's power limit, and the bytes moved from L2 into shared memory per flop are
// the part of that budget a kernel can shrink (with constant operand bits this kernel's K loop
// reaches 91 % of the tensor pipe's own rate) -- and the
// 512 TMEM columns are exactly used up: 384 accumulator + 4 x 32 scale columns.  Every CTA
// fetches its own operands with plain TMA loads; only barrier signals cross the pair.
//
// Roles per CTA (512 threads, four warpgroups; registers rebalanced with setmaxnreg):
//   warps 0..3   scale warps (one per TMEM lane quadrant): shared memory -> this CTA's TMEM scale
//                columns with tcgen05.st.  (tcgen05.cp would do the same copy, but measured here
//                each one holds the tensor pipe for 70-85 cycles whatever its shape, and a
//                K-step needs eight of them against 768 cycles of MMA.)
//   warps 4..11  epilogue: this CTA's 128 rows x 384 columns of the accumulator, 32 rows x 192
//                columns per warp in two rounds of three tcgen05.ld; the accumulator is handed
//                back as soon as the second round has landed, then alpha, conversion and stores
//                overlap the next tile's main loop.
//   warp 12      TMA producer: A half and two B sub-tiles (completion counted on the LEADER's
//                barrier) and the scale tiles (local barrier), 4-stage ring.
//   warp 13      MMA issuer, leader CTA (cluster rank 0) only: eight
//                tcgen05.mma.cta_group::2.kind::mxf4.block_scale (256 x 192 x 64) per stage; its
//                commits arrive on the barriers of both CTAs.
// The issuing warps run their loops in warp-uniform control flow and issue through
// elect.sync, so descriptors stay in uniform registers; the MMA warp tests the next stage's
// barriers before it issues the current stage's MMAs, which hides the barrier round trip.
// Barrier ownership: full / sf_ready / tmem_empty are consumed by the leader's MMA warp, so the
// peer's producer, scale warps and epilogue warps arrive on the leader's copies (relaxed: they
// publish no ordinary memory writes); empty and tmem_full are signalled in both CTAs by a
// multicast tcgen05.commit; sf_full is local.  All waits are bounded (see ptx_sm100.cuh).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <mutex>

#include "../../include/mxfp4.h"
#include "ptx_sm100.cuh"
#include "tma_host.cuh"

namespace mxfp4 {

constexpr int kPHalfM = 128;                     // rows of A (and of the accumulator) per CTA
constexpr int kPTileM = 256;
constexpr int kPTileN = 384;                     // two MMAs of N = 192 per K = 64
constexpr int kPMmaN = 192;
constexpr int kPSubN = 96;                       // rows of B per CTA per MMA
constexpr int kPBlockK = 256;                    // elements per stage = 128 bytes of codes per row
constexpr int kPStages = 4;
constexpr int kPABytes = kPHalfM * 128;          // 16 KB
constexpr int kPBSubBytes = kPSubN * 128;        // 12 KB
constexpr int kPSfaBytes = 2 * 512;              // own 128 rows x 2 K-tiles of 128 elements
constexpr int kPSfbBytes = 3 * 2 * 512;          // three 128-row blocks of B x 2 K-tiles
constexpr int kPEpiWarps = 8;
constexpr int kPProducerWarp = 12;
constexpr int kPMmaWarp = 13;
constexpr int kPThreads = 512;
constexpr uint32_t kPTmemCols = 512;
constexpr uint32_t kPTmemSfBase = 384;           // accumulator occupies columns 0..383
constexpr uint32_t kPTmemSfPerBuf = 32;          // per stage: 8 columns SFA + 24 columns SFB

struct GemmPairSmem {
    alignas(1024) uint8_t a[kPStages][kPABytes];          // 128 rows x 128 B
    alignas(1024) uint8_t b[kPStages][2][kPBSubBytes];    // [MMA half][96 rows x 128 B]
    alignas(128) uint8_t sfa[kPStages][kPSfaBytes];       // [K-tile][512]
    alignas(128) uint8_t sfb[kPStages][kPSfbBytes];       // [row block][K-tile][512]
    alignas(1024) uint8_t out_stage[kPEpiWarps][32 * 128]; // 32 rows x 64 bf16 per warp, 128-byte swizzle
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
    int32_t tiles_m, tiles_n;   // 256 x 384 pair tiles
    int32_t band_m;             // tile rows per band of the tile order (see gemm_tile_coords)
    int32_t band_n;             // 0, or tile columns per band when the bands run along N instead
    int32_t k_stages;           // ceil(K / 256)
    int32_t sf_tiles_k;         // ceil(K / 128)
    int32_t sf_rows_a;          // ceil(M / 128)
    int32_t sf_rows_b;          // ceil(N / 128)
    float alpha;
    int32_t out_fp32;
    int32_t n_tma;              // columns written by TMA stores: N rounded down to a 16-byte granule (8 bf16 / 4 fp32)
};

// Instruction descriptor of the pair MMA: E2M1 x E2M1, E8M0 scales, both operands K-major,
// M = 256 (128 per CTA), N = 192.  Scale-factor ids select which byte pair of the 32-bit TMEM
// scale column an instruction uses.
// KIND 1 (8-bit operands): E4M3 x E4M3, whose format code under kind::mxf8f6f4 is 0, and the
// scale-factor id selects one byte of the column.
template <int KIND>
__device__ __forceinline__ uint32_t make_idesc_mx_pair(uint32_t a_sf_id, uint32_t b_sf_id)
{
    uint32_t d = 0;
    d |= b_sf_id << 4;                 // bits 4..5   B scale-factor id
    d |= (KIND == 0 ? 1u : 0u) << 7;   // bits 7..9   A format: E2M1 (mxf4) / E4M3 (mxf8f6f4)
    d |= (KIND == 0 ? 1u : 0u) << 10;  // bits 10..12 B format
    //                                    bits 17..22 N / 8: added per MMA (idesc_n), see below
    d |= 1u << 23;                     // bit 23      scale format: E8M0
    d |= (kPTileM >> 4) << 24;         // bits 24..28 M / 16
    d |= a_sf_id << 29;                // bits 29..30 A scale-factor id
    return d;
}

// N field of the instruction descriptor.  N is 192 for every MMA except in a matrix's last tile
// column, where it shrinks to the columns that exist (rounded up to the instruction's granule of
// 16): an MMA's issue time is proportional to N, so e.g. the 256 columns that N = 4096 leaves for
// its eleventh tile cost 192 + 64 instead of 2 x 192.
__device__ __forceinline__ uint32_t idesc_n(int n) { return static_cast<uint32_t>(n >> 3) << 17; }

// Tile order.  The persistent clusters take tiles cluster_id, cluster_id + n_clusters, ..., so at any
// time about n_clusters consecutive tiles are in flight and read the same K range of their A and B
// panels.  Tiles are numbered band by band: a band is `band_m` tile rows of M, and inside a band the
// tile row varies fastest, then the tile column.  The A panel of a band (band_m x 256 rows x K) is
// sized by the host to stay in L2 while the band sweeps across N, so A comes from HBM once; B is
// re-read once per band.  (With a single band -- every shape whose A fits in L2 -- this is plain
// column-major order.  With tile rows fastest over ALL of M, a long-K A that exceeds L2 was
// streamed from HBM once per tile column: 2.6 GB instead of 0.7 GB for 16384 x 4096 x 28672.)
// When B is the smaller panel the bands run along N instead (`band_n` > 0): a band is `band_n` tile
// columns whose B panel stays in L2, inside a band the tile column varies fastest, so that all of a
// tile row's columns are in flight together and A streams from HBM once per band.
__device__ __forceinline__ void gemm_tile_coords(const GemmPairParams& p, int tile, int& tm, int& tn)
{
    if (p.band_n > 0) {
        const int per_band = p.band_n * p.tiles_m;
        const int band = tile / per_band;
        const int r = tile - band * per_band;
        const int cols = min(p.band_n, p.tiles_n - band * p.band_n);    // the last band may be narrower
        tm = r / cols;
        tn = band * p.band_n + (r - tm * cols);
        return;
    }
    const int per_band = p.band_m * p.tiles_n;
    const int band = tile / per_band;
    const int r = tile - band * per_band;
    const int rows = min(p.band_m, p.tiles_m - band * p.band_m);    // the last band may be shorter
    tn = r / rows;
    tm = band * p.band_m + (r - tn * rows);
}

// Columns the two MMAs of a tile in tile column `tn` compute: n0 for accumulator columns 0..191,
// n1 (possibly 0: no MMA) for columns 192..383.  CTA r of the pair supplies rows
// [r * n / 2, (r + 1) * n / 2) of the MMA's n rows of B, so the producer needs the same numbers.
__device__ __forceinline__ void tile_mma_widths(int N, int tn, int& n0, int& n1)
{
    const int nv = min(kPTileN, N - tn * kPTileN);
    n0 = min(kPMmaN, (nv + 15) & ~15);
    n1 = nv > kPMmaN ? min(kPMmaN, (nv - kPMmaN + 15) & ~15) : 0;
}

// The kernel body for both operand widths.  A stage is 128 bytes of codes per operand row either
// way -- 256 four-bit or 128 eight-bit elements -- and four MMA K-steps of 32 bytes, so the
// pipeline, the tile shape and the epilogue are shared; what differs is the instruction kind,
// the number of 128-element scale tiles a stage covers (two / one) and how an MMA addresses its
// scales (a byte pair of one of two columns / one byte of one column).
template <int KIND>
__device__ __forceinline__ void gemm_pair_body(const CUtensorMap& tm_a, const CUtensorMap& tm_b,
                                               const CUtensorMap& tm_out, const GemmPairParams& p)
{
    constexpr int kBlockK = KIND == 0 ? kPBlockK : kPBlockK / 2;   // elements per stage
    constexpr int kMmaK = KIND == 0 ? 64 : 32;                     // elements per MMA
    constexpr int kSfTilesPerStage = KIND == 0 ? 2 : 1;
    extern __shared__ uint8_t smem_raw[];
    GemmPairSmem& sm = *reinterpret_cast<GemmPairSmem*>(smem_align_1024(smem_raw));
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
    // set-up done: let the next kernel's CTAs take SMs as they free up, and do not touch global
    // memory before the previous kernel in the stream has completed
    griddep_launch_dependents();
    griddep_wait();

    // register budget per role (whole warpgroups): 4*32*(56 + 2*192 + 72) = 65536, all of the register
    // file; every warp of a warpgroup executes the same setmaxnreg at the top of its role
    if (warp == kPProducerWarp) {
        // ------------------------------------------------------------ TMA producer
        setmaxnreg_dec<72>();
        if (lane == 0) {
            tma_prefetch_desc(&tm_a);
            tma_prefetch_desc(&tm_b);
        }
        int it = 0;
        bool alive = true;
        for (int t = 0; alive && t < my_tiles; ++t) {
            const int tile = cluster_id + t * n_clusters;
            int tm, tn;
            gemm_tile_coords(p, tile, tm, tn);
            const int a_row_tile = tm * 2 + static_cast<int>(rank);     // 128-row scale tile of A
            int n0, n1;
            tile_mma_widths(p.N, tn, n0, n1);
            // this CTA's share of B: rows [rank * n / 2, ...) of each MMA's n rows (the box is always 96
            // rows: what lies beyond the share is not read by the MMA, what lies beyond N arrives as zeros)
            const int32_t yb0 = tn * kPTileN + static_cast<int>(rank) * (n0 >> 1);
            const int32_t yb1 = tn * kPTileN + kPMmaN + static_cast<int>(rank) * (n1 >> 1);
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
                    mbar_arrive_expect_tx_cluster(full_leader, kPABytes + 2 * kPBSubBytes);
                    const int32_t x = ks * 128;                          // bytes along the code row
                    const int32_t ya = tm * kPTileM + rank * kPHalfM;
                    tma_load_2d_pair(sm.a[s], &tm_a, full_leader, x, ya);
                    tma_load_2d_pair(sm.b[s][0], &tm_b, full_leader, x, yb0);
                    tma_load_2d_pair(sm.b[s][1], &tm_b, full_leader, x, yb1);
                    // scales: local barrier
                    const int kt0 = ks * kSfTilesPerStage;
                    const int nkt = min(kSfTilesPerStage, p.sf_tiles_k - kt0);
                    const uint32_t sf_bytes = nkt * 512;
                    const int has_a = a_row_tile < p.sf_rows_a ? 1 : 0;
                    const int nb0 = tn * 3;
                    const int nnb = max(0, min(3, p.sf_rows_b - nb0));
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
    } else if (warp == kPMmaWarp) {
        // ------------------------------------------------------------ MMA issuer (leader only)
        setmaxnreg_dec<72>();
        if (rank == 0 && total_it > 0) {
            int it = 0;
            bool alive = true;
            // readiness of the current stage as seen by the test issued one stage earlier
            bool rdy_full = false, rdy_sf = false;
            // descriptors of stage 0; a stage adds a constant, a K = 64 step adds 32 bytes
            const uint64_t a_desc0 = make_smem_desc(smem_u32(sm.a[0]), 16, 1024, 2);
            const uint64_t b_desc0 = make_smem_desc(smem_u32(sm.b[0][0]), 16, 1024, 2);
            // scale-factor ids by K-step: byte pairs 0 / 2 of alternating columns (4-bit), bytes 0..3 (8-bit)
            const uint32_t idesc0 = make_idesc_mx_pair<KIND>(0, 0), idesc2 = make_idesc_mx_pair<KIND>(2, 2);
            const uint32_t idesc1 = make_idesc_mx_pair<KIND>(1, 1), idesc3 = make_idesc_mx_pair<KIND>(3, 3);
            int s = 0;
            uint32_t parity = 0;
            for (int tile_it = 0; alive && tile_it < my_tiles; ++tile_it) {
                int n0, n1, tm_unused, tn;
                gemm_tile_coords(p, cluster_id + tile_it * n_clusters, tm_unused, tn);
                tile_mma_widths(p.N, tn, n0, n1);
                const uint32_t idn0 = idesc_n(n0), idn1 = idesc_n(n1);
                if (tile_it > 0 && !mbar_wait(&sm.tmem_empty, (tile_it - 1) & 1, &sm.abort_flag)) break;
                for (int ks = 0; ks < p.k_stages; ++ks, ++it) {
                    // codes landed in both CTAs' shared memory; scales landed in both CTAs' TMEM
                    if ((!rdy_full && !mbar_wait(&sm.full[s], parity, &sm.abort_flag)) ||
                        (!rdy_sf && !mbar_wait(&sm.sf_ready[s], parity, &sm.abort_flag))) {
                        alive = false;
                        break;
                    }
                    tcgen05_fence_after();
                    const int s1 = (s + 1 == kPStages) ? 0 : s + 1;
                    const uint32_t parity1 = (s + 1 == kPStages) ? parity ^ 1u : parity;
                    if (it + 1 < total_it) {
                        rdy_full = mbar_test_wait(&sm.full[s1], parity1);
                        rdy_sf = mbar_test_wait(&sm.sf_ready[s1], parity1);
                    }
                    const uint32_t sf_tmem = tmem + kPTmemSfBase + s * kPTmemSfPerBuf;
                    const int valid_k = min(kBlockK, p.K - ks * kBlockK);
                    const int nmma = (valid_k + kMmaK - 1) / kMmaK;
                    if (elect_one_sync()) {
                        const uint64_t a_desc = a_desc0 + static_cast<uint64_t>(s * (kPABytes >> 4));
                        const uint64_t b_desc = b_desc0 + static_cast<uint64_t>(s * ((2 * kPBSubBytes) >> 4));
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            if (j < nmma) {
                                // K-step j: 32 bytes along the 128-byte swizzled row; two MMAs, one per
                                // 192-column half of the tile
                                const uint32_t idesc = KIND == 0 ? ((j & 1) ? idesc2 : idesc0)
                                                                 : (j == 0 ? idesc0 : j == 1 ? idesc1 : j == 2 ? idesc2 : idesc3);
                                const uint32_t sfa = sf_tmem + (KIND == 0 ? (j >> 1) * 4 : 0);
                                const uint32_t sfb = sf_tmem + 8 + (KIND == 0 ? (j >> 1) * 12 : 0);
                                tcgen05_mma_mx_pair_collect<KIND, 0>(tmem, a_desc + 2 * j, b_desc + 2 * j, idesc | idn0, sfa,
                                                                     sfb, (ks > 0 || j > 0) ? 1u : 0u);
                                if (n1 > 0)
                                    tcgen05_mma_mx_pair_collect<KIND, 1>(tmem + kPMmaN, a_desc + 2 * j,
                                                                         b_desc + 2 * j + (kPBSubBytes >> 4), idesc | idn1,
                                                                         sfa, sfb + 6, (ks > 0 || j > 0) ? 1u : 0u);
                            }
                        }
                        // frees the shared-memory stage and its TMEM scale columns in both CTAs
                        tcgen05_commit_pair(&sm.empty[s], 3);
                    }
                    __syncwarp();
                    s = s1;
                    parity = parity1;
                }
                if (alive && elect_one_sync()) tcgen05_commit_pair(&sm.tmem_full, 3);
                __syncwarp();
            }
        }
    } else if (warp < 4) {
        // ------------------------------------------------------------ scale warps
        // Lane r of every quadrant must hold, per 128-row x 4-block scale tile, the 16 bytes at
        // offset 16*r of that tile: four 32-bit columns = rows r, r+32, r+64, r+96.  Stage s
        // owns TMEM columns [s*32, s*32+32): SFA K-tiles 0,1 (4 columns each) | SFB K-tile 0
        // (12 columns: row blocks 0,1,2) | SFB K-tile 1.  The columns are free again once the
        // producer has seen empty[s], which happens before sf_full[s] can complete.
        setmaxnreg_dec<56>();
        const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
        const uint32_t sf_ready_leader_base = map_to_cta(smem_u32(&sm.sf_ready[0]), 0);
        for (int it = 0; it < total_it; ++it) {
            const int s = it % kPStages;
            if (!mbar_wait(&sm.sf_full[s], (it / kPStages) & 1, &sm.abort_flag)) break;
            const uint32_t t = tmem + lane_base + kPTmemSfBase + s * kPTmemSfPerBuf;
            const uint8_t* sa = &sm.sfa[s][lane * 16];
            const uint8_t* sb = &sm.sfb[s][lane * 16];           // [row block nb][K-tile kt] at nb*1024 + kt*512
            auto lda = [&](const uint8_t* q) { return smem_load<uint4>(q, sm.sfa[s], kPSfaBytes); };
            auto ldb = [&](const uint8_t* q) { return smem_load<uint4>(q, sm.sfb[s], kPSfbBytes); };
            tmem_st_32x32b_x8(t, lda(sa), lda(sa + 512));                       // SFA kt0 | kt1
            tmem_st_32x32b_x8(t + 8, ldb(sb), ldb(sb + 1024));                  // SFB kt0: nb0 | nb1
            tmem_st_32x32b_x8(t + 16, ldb(sb + 2048), ldb(sb + 512));           // SFB kt0: nb2 | kt1: nb0
            tmem_st_32x32b_x8(t + 24, ldb(sb + 1024 + 512), ldb(sb + 2048 + 512));  // SFB kt1: nb1 | nb2
            tmem_st_wait();
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(sf_ready_leader_base + s * 8);
        }
    } else if (warp < 12) {
        // ------------------------------------------------------------ epilogue warps
        setmaxnreg_inc<192>();
        const int ew = warp - 4;
        const int quad = warp & 3;                 // TMEM lane quadrant this warp may read
        const int half = ew >> 2;                  // which 192 accumulator columns
        uint8_t* stg = sm.out_stage[ew];
        const uint64_t store_policy = l2_policy_evict_first();   // the output streams out once
        const uint32_t tmem_empty_leader = map_to_cta(smem_u32(&sm.tmem_empty), 0);
        for (int tile_it = 0; tile_it < my_tiles; ++tile_it) {
            const int tile = cluster_id + tile_it * n_clusters;
            int tm, tn;
            gemm_tile_coords(p, tile, tm, tn);
            if (!mbar_wait(&sm.tmem_full, tile_it & 1, &sm.abort_flag)) break;
            tcgen05_fence_after();
            const uint32_t taddr = tmem + (static_cast<uint32_t>(quad * 32) << 16) + half * kPMmaN;
            const int64_t row0 = static_cast<int64_t>(tm) * kPTileM + rank * kPHalfM + quad * 32;
            const int64_t colbase = static_cast<int64_t>(tn) * kPTileN + half * kPMmaN;
            if (p.out_fp32) {
                // fp32 output: two rounds of 96 columns; TMEM is released after the second load
                const int64_t row = row0 + lane;
#pragma unroll
                for (int round = 0; round < 2; ++round) {
                    uint32_t r[3][32];
#pragma unroll
                    for (int c = 0; c < 3; ++c) tmem_ld_32x32b_x32(taddr + round * 96 + c * 32, r[c]);
                    tmem_ld_wait();
                    if (round == 1) {
                        tcgen05_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(tmem_empty_leader);
                    }
                    // three passes of 32 columns: the warp lays its 32 rows x 128 bytes out in the
                    // 128-byte swizzle and one lane hands the box to a TMA store, as for bf16
#pragma unroll
                    for (int c = 0; c < 3; ++c) {
                        const int64_t col0 = colbase + round * 96 + c * 32;
                        if (lane == 0) bulk_wait_group_read<0>();
                        __syncwarp();
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            smem_store(stg + lane * 128 + ((q ^ (lane & 7)) * 16),
                                       make_float4(__uint_as_float(r[c][4 * q]) * p.alpha,
                                                   __uint_as_float(r[c][4 * q + 1]) * p.alpha,
                                                   __uint_as_float(r[c][4 * q + 2]) * p.alpha,
                                                   __uint_as_float(r[c][4 * q + 3]) * p.alpha),
                                       stg, 32 * 128);
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (p.n_tma < p.N) {
                            // N is not a multiple of 4: the tensor map ends at the last full 16-byte
                            // granule; the one to three columns after it come from the staged row
                            const int64_t rc = p.n_tma - col0;
                            if (rc >= 0 && rc < 32 && row < p.M) {
                                const int q = static_cast<int>(rc >> 2);
                                const float4 v = smem_load<float4>(stg + lane * 128 + ((q ^ (lane & 7)) * 16), stg, 32 * 128);
                                const float e[4] = {v.x, v.y, v.z, v.w};
                                float* dst = static_cast<float*>(p.out) + row * p.ld_out + p.n_tma;
                                for (int k = 0; k < 3; ++k)
                                    if (p.n_tma + k < p.N) dst[k] = e[k];
                            }
                        }
                        if (lane == 0 && row0 < p.M && col0 < p.n_tma) {
                            tma_store_2d_hint(&tm_out, stg, static_cast<int32_t>(col0), static_cast<int32_t>(row0),
                                              store_policy);
                            bulk_commit_group();
                        }
                    }
                }
            } else {
                // bf16 output: 192 columns of this thread's row as 96 packed words; the first 96
                // columns are converted while the second 96 are still in flight, and TMEM is
                // released before any store
                uint32_t w[96];
#pragma unroll
                for (int round = 0; round < 2; ++round) {
                    uint32_t r[3][32];
#pragma unroll
                    for (int c = 0; c < 3; ++c) tmem_ld_32x32b_x32(taddr + round * 96 + c * 32, r[c]);
                    tmem_ld_wait();
                    if (round == 1) {
                        tcgen05_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(tmem_empty_leader);
                    }
#pragma unroll
                    for (int c = 0; c < 3; ++c)
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(r[c][2 * i]) * p.alpha,
                                                                           __uint_as_float(r[c][2 * i + 1]) * p.alpha);
                            w[round * 48 + c * 16 + i] = *reinterpret_cast<const uint32_t*>(&v);
                        }
                }
                // three passes of 64 columns: the warp lays its 32 rows x 128 bytes out in the
                // 128-byte swizzle and one lane hands the box to a TMA store (which clips at the
                // matrix edges); the buffer is reused once the previous store has read it
#pragma unroll
                for (int c = 0; c < 3; ++c) {
                    if (lane == 0) bulk_wait_group_read<0>();
                    __syncwarp();
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        smem_store(stg + lane * 128 + ((q ^ (lane & 7)) * 16),
                                   make_uint4(w[c * 32 + q * 4], w[c * 32 + q * 4 + 1], w[c * 32 + q * 4 + 2],
                                              w[c * 32 + q * 4 + 3]),
                                   stg, 32 * 128);
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (p.n_tma < p.N) {
                        // N is not a multiple of 8: a TMA store writes whole 16-byte granules, so
                        // the tensor map ends at the last full granule and the few columns after
                        // it are stored one by one from this thread's staged row
                        const int64_t rc = p.n_tma - (colbase + c * 64);
                        const int64_t row = row0 + lane;
                        if (rc >= 0 && rc < 64 && row < p.M) {
                            const int q = static_cast<int>(rc >> 3);
                            const uint4 v = smem_load<uint4>(stg + lane * 128 + ((q ^ (lane & 7)) * 16), stg, 32 * 128);
                            const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&v);
                            __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(p.out) + row * p.ld_out + p.n_tma;
                            for (int k = 0; k < 8; ++k)
                                if (p.n_tma + k < p.N) dst[k] = e[k];
                        }
                    }
                    if (lane == 0 && row0 < p.M && colbase + c * 64 < p.n_tma) {
                        tma_store_2d_hint(&tm_out, stg, static_cast<int32_t>(colbase + c * 64),
                                          static_cast<int32_t>(row0), store_policy);
                        bulk_commit_group();
                    }
                }
            }
        }
        if (lane == 0) bulk_wait_group<0>();
    } else {
        setmaxnreg_dec<72>();   // idle warps of the producer/MMA warpgroup
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

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPThreads, 1)
gemm_mxf4_pair_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                      const __grid_constant__ CUtensorMap tm_out, const GemmPairParams p)
{
    gemm_pair_body<0>(tm_a, tm_b, tm_out, p);
}

// The 8-bit GEMM of the passes the precision ladder leaves in FP8 (Table 1): E4M3 codes, one
// byte per element, the same tiled E8M0 scales.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPThreads, 1)
gemm_mxf8_pair_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                      const __grid_constant__ CUtensorMap tm_out, const GemmPairParams p)
{
    gemm_pair_body<1>(tm_a, tm_b, tm_out, p);
}

template <int KIND>
static int launch_gemm_pair(const void* a_codes, const void* a_scales, const void* b_codes,
                            const void* b_scales, int64_t M, int64_t N, int64_t K, float alpha, void* out,
                            int out_dtype, int64_t ld_out, int sm_count, cudaStream_t stream)
{
    CUtensorMap tm_a, tm_b, tm_out;
    // output through TMA stores of 128-byte x 32-row boxes: 64 bf16 or 32 fp32 columns
    const bool bf16_out = out_dtype == MXFP4_OUT_BF16;
    const int64_t n_tma = bf16_out ? (N & ~static_cast<int64_t>(7)) : (N & ~static_cast<int64_t>(3));
    if (n_tma > 0) {
        if (!make_tmap_2d(&tm_out, bf16_out ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                          bf16_out ? 2 : 4, out, M, n_tma, ld_out * (bf16_out ? 2 : 4), 32, bf16_out ? 64 : 32,
                          CU_TENSOR_MAP_SWIZZLE_128B))
            return MXFP4_ERR_CUDA;
    } else {
        memset(&tm_out, 0, sizeof(tm_out));
    }
    // codes as bytes: [rows x K/2] (4-bit) or [rows x K] (8-bit), boxes of 128 bytes x 128 rows (A) /
    // 96 rows (B), 128-byte swizzle
    const int64_t row_bytes = KIND == 0 ? K / 2 : K;
    if (!make_tmap_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a_codes, M, row_bytes, row_bytes, kPHalfM, 128,
                      CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, b_codes, N, row_bytes, row_bytes, kPSubN, 128,
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
    {
        // band height of the tile order: as many tile rows as keep the band's A panel within about a
        // quarter of the L2 (32 MB), so that it survives the band's sweep across N beside the B
        // panels streaming through
        const int64_t row_b = KIND == 0 ? K / 2 : K;                     // bytes of codes per operand row
        const int64_t a_tile_row_bytes = static_cast<int64_t>(kPTileM) * row_b;
        int64_t band = (32ll << 20) / (a_tile_row_bytes > 0 ? a_tile_row_bytes : 1);
        if (band < 1) band = 1;
        if (band > p.tiles_m) band = p.tiles_m;
        p.band_m = static_cast<int32_t>(band);
        // the same along N (a few MB more of budget, so that eleven tile columns of a 4096-wide B make
        // one or two bands); the orientation with the smaller estimate of HBM reads wins (bands along
        // M read A once and B once per band, bands along N the other way round); a tie -- both panels
        // fit, one band either way -- goes to N, 1-2 % faster on the 4096 x 4096 projections
        const int64_t b_tile_col_bytes = static_cast<int64_t>(kPTileN) * row_b;
        int64_t band_n = (36ll << 20) / (b_tile_col_bytes > 0 ? b_tile_col_bytes : 1);
        if (band_n < 1) band_n = 1;
        if (band_n > p.tiles_n) band_n = p.tiles_n;
        const int64_t bands_m = (p.tiles_m + band - 1) / band, bands_n = (p.tiles_n + band_n - 1) / band_n;
        const int64_t a_bytes = M * row_b, b_bytes = N * row_b;
        const int64_t cost_m = a_bytes + b_bytes * bands_m, cost_n = b_bytes + a_bytes * bands_n;
        p.band_n = cost_n <= cost_m ? static_cast<int32_t>(band_n) : 0;
    }
    constexpr int kBlockK = KIND == 0 ? kPBlockK : kPBlockK / 2;
    p.k_stages = static_cast<int32_t>((K + kBlockK - 1) / kBlockK);
    p.sf_tiles_k = static_cast<int32_t>((K + 127) / 128);
    p.sf_rows_a = static_cast<int32_t>((M + 127) / 128);
    p.sf_rows_b = static_cast<int32_t>((N + 127) / 128);
    p.alpha = alpha;
    p.out_fp32 = out_dtype == MXFP4_OUT_FP32;
    p.n_tma = static_cast<int32_t>(n_tma);
    const int64_t total = static_cast<int64_t>(p.tiles_m) * p.tiles_n;
    if (total > 0x3FFFFFFF) return MXFP4_ERR_SHAPE;
    const size_t smem = sizeof(GemmPairSmem) + 1024;
    // per device, set up once however many host threads arrive together: the shared-memory
    // attribute and the number of CTA pairs that can be resident at once
    static int resident_clusters[64] = {};
    static std::once_flag once[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MXFP4_ERR_CUDA;
    std::call_once(once[dev], [&] {
        auto kernel = KIND == 0 ? gemm_mxf4_pair_kernel : gemm_mxf8_pair_kernel;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) !=
            cudaSuccess)
            return;                                     // resident_clusters stays 0: reported below
        // the persistent grid must not exceed what the device can hold at once (a partitioned or
        // shared device may offer fewer pairs than SMs / 2); fall back to SMs / 2 if the query fails
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(sm_count & ~1), 1, 1);
        cfg.blockDim = dim3(kPThreads, 1, 1);
        cfg.dynamicSmemBytes = smem;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess || n <= 0) {
            (void)cudaGetLastError();
            n = sm_count / 2;
        }
        resident_clusters[dev] = n < sm_count / 2 ? n : sm_count / 2;
    });
    if (resident_clusters[dev] <= 0) return MXFP4_ERR_CUDA;
    const int max_clusters = resident_clusters[dev];
    const int clusters = static_cast<int>(total < max_clusters ? total : max_clusters);
    return launch_kernel_pdl(KIND == 0 ? gemm_mxf4_pair_kernel : gemm_mxf8_pair_kernel, 2 * clusters, kPThreads, smem,
                             stream, tm_a, tm_b, tm_out, p) == cudaSuccess
               ? MXFP4_OK : MXFP4_ERR_CUDA;
}

}  // namespace mxfp4
