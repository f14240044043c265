// Thin inline-PTX wrappers for sm_100a: mbarrier, TMA (cp.async.bulk[.tensor]), tcgen05
// (TMEM allocation, MMA, commit, ld, st) and the bounded-wait discipline every kernel of this
// library follows: no wait spins forever; a wait that runs out records a status word and
// makes every later wait of the CTA return at once.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace mxfp4 {

// Sticky device-side status (0 = OK).  Written with atomicCAS so the first error wins.
// The library is a single translation unit, so the definition lives here.
__device__ int g_device_status = 0;

constexpr int kDevErrTimeout = -7;
constexpr int kDevErrBounds = -10;

// Bounds discipline of the debug build (-DMXFP4_BOUNDS), the stand-in for a memory sanitizer: every
// access whose address a kernel COMPUTES (shared-memory stages, staging tiles, scale tiles) goes
// through smem_load / smem_store, which in that build check that the address lies inside the
// buffer it was derived from and is naturally aligned; a miss records kDevErrBounds in the status
// word and the access is skipped (a load returns zeros) -- nothing traps.  In the normal build the
// helpers are plain loads and stores.
__device__ __forceinline__ bool bounds_ok(const void* p, size_t bytes, const void* base, size_t size)
{
    const uintptr_t a = reinterpret_cast<uintptr_t>(p), b = reinterpret_cast<uintptr_t>(base);
    if (a >= b && a + bytes <= b + size && a % bytes == 0) return true;
    atomicCAS(&g_device_status, 0, kDevErrBounds);
    return false;
}

template <class T>
__device__ __forceinline__ T smem_load(const void* p, const void* base, size_t size)
{
#ifdef MXFP4_BOUNDS
    if (!bounds_ok(p, sizeof(T), base, size)) return T{};
#endif
    return *static_cast<const T*>(p);
}

template <class T>
__device__ __forceinline__ void smem_store(void* p, const T& v, const void* base, size_t size)
{
#ifdef MXFP4_BOUNDS
    if (!bounds_ok(p, sizeof(T), base, size)) return;
#endif
    *static_cast<T*>(p) = v;
}

// Spin limit for one wait.  A try_wait suspends for a hardware-defined slice, so this many
// attempts is on the order of a second -- far longer than any legitimate wait here.
constexpr uint32_t kSpinLimit = 1u << 20;

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// Start of a kernel's dynamic shared memory rounded up to 1024 bytes (what the 128-byte swizzle
// wants).  The padding is added to the POINTER: rounding the address up as an integer and casting
// back hides the address space from the compiler, and every access through such a pointer becomes
// a generic load or store (global-path latency, 64-bit address arithmetic) instead of
// ld.shared / st.shared.
__device__ __forceinline__ uint8_t* smem_align_1024(uint8_t* smem_raw)
{
    return smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
}

// The same address reached through an integer: accesses through the result are generic loads and
// stores.  Kept for the one kernel variant that measures faster that way (see quantize_dual_kernel).
__device__ __forceinline__ uint8_t* smem_align_1024_generic(uint8_t* smem_raw)
{
    return reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
}

// Programmatic dependent launch: every kernel of the library is launched with the
// programmatic-stream-serialization attribute, so its CTAs may start (barrier set-up, TMEM
// allocation, descriptor prefetch) while the previous kernel in the stream is still draining.
// griddep_wait() returns once that previous kernel has completed and its writes are visible;
// every kernel executes it before its first global-memory access, which keeps stream order
// transitive.  griddep_launch_dependents() lets the next kernel's CTAs be scheduled as soon as
// SMs free up.  Both are no-ops for a kernel launched without the attribute.
__device__ __forceinline__ void griddep_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ void griddep_launch_dependents()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

__device__ __forceinline__ uint32_t elect_one_sync()
{
    uint32_t pred = 0;
    asm volatile(
        "{\n\t.reg .pred P;\n\t"
        "elect.sync _|P, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, P;\n\t}"
        : "=r"(pred));
    return pred;
}

// ---------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}

__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred P;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 P, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, P;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Non-blocking test of a barrier phase (never suspends the thread).
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred P;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 P, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, P;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait.  `abort_flag` is a CTA-shared word: once set, waits return immediately so the
// CTA drains and exits.  Returns false if the wait was abandoned.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          uint32_t spin_limit = kSpinLimit)
{
    for (uint32_t spin = 0; spin < spin_limit; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    atomicCAS(&g_device_status, 0, kDevErrTimeout);
    return false;
}

// ---------------------------------------------------------------- async-proxy fences
__device__ __forceinline__ void fence_proxy_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---------------------------------------------------------------- TMA
__device__ __forceinline__ void tma_prefetch_desc(const void* tmap)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tmap)) : "memory");
}

// 2-D tiled load global -> shared, completion counted in bytes on `bar`.  x is the
// innermost coordinate (x * element size must be a multiple of 16 bytes).
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const void* tmap, uint64_t* bar,
                                            int32_t x, int32_t y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(smem_u32(bar)),
        "r"(x), "r"(y)
        : "memory");
}

// 2-D tiled prefetch global -> L2: the box a later tma_load_2d will fetch, so that load finds its
// data in L2 (same alignment rule for x).
__device__ __forceinline__ void tma_prefetch_l2_2d(const void* tmap, int32_t x, int32_t y)
{
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global [%0, {%1, %2}];"
                 ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y)
                 : "memory");
}

// 2-D tiled store shared -> global (bulk async-group completion).
__device__ __forceinline__ void tma_store_2d(const void* tmap, const void* smem_src, int32_t x,
                                             int32_t y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
        ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(smem_u32(smem_src)), "r"(x), "r"(y)
        : "memory");
}

// L2 eviction-priority policies for cache-hinted TMA traffic.
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

// 2-D tiled store with an L2 cache hint (streaming outputs should not displace operands).
__device__ __forceinline__ void tma_store_2d_hint(const void* tmap, const void* smem_src, int32_t x,
                                                  int32_t y, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;"
        ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(smem_u32(smem_src)), "r"(x), "r"(y), "l"(policy)
        : "memory");
}

// 1-D bulk copies (addresses 16-byte aligned, size a multiple of 16).
__device__ __forceinline__ void bulk_load_1d(void* smem_dst, const void* gsrc, uint32_t bytes,
                                             uint64_t* bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(gsrc)), "r"(bytes),
        "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void bulk_store_1d(void* gdst, const void* smem_src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(reinterpret_cast<uint64_t>(gdst)), "r"(smem_u32(smem_src)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void bulk_commit_group()
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

template <int N>
__device__ __forceinline__ void bulk_wait_group_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}

template <int N>
__device__ __forceinline__ void bulk_wait_group()
{
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}

// ---------------------------------------------------------------- tcgen05 / TMEM
__device__ __forceinline__ void tcgen05_fence_before()
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}

__device__ __forceinline__ void tcgen05_fence_after()
{
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// 32 lanes x 32 consecutive 32-bit columns -> 32 registers per thread (lane = thread's row).
__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
          "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
          "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]),
          "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]),
          "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

// 32 lanes x 8 consecutive 32-bit columns <- 8 registers per thread (lane = thread's row).
__device__ __forceinline__ void tmem_st_32x32b_x8(uint32_t taddr, const uint4& lo, const uint4& hi)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"r"(taddr), "r"(lo.x), "r"(lo.y), "r"(lo.z), "r"(lo.w), "r"(hi.x), "r"(hi.y),
                 "r"(hi.z), "r"(hi.w)
                 : "memory");
}

__device__ __forceinline__ void tmem_st_wait()
{
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// Per-warpgroup register rebalancing (all four warps of a warpgroup execute the same one).
template <int N>
__device__ __forceinline__ void setmaxnreg_inc()
{
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}

template <int N>
__device__ __forceinline__ void setmaxnreg_dec()
{
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

__device__ __forceinline__ void tmem_ld_wait()
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor (K-major operand).  Fields: start address >> 4 in bits
// 0..13, leading byte offset >> 4 in 16..29, stride byte offset >> 4 in 32..45, descriptor
// version 1 in 46..47, swizzle mode in 61..63 (0 none, 2 = 128 B, 4 = 64 B, 6 = 32 B).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr, uint32_t lbo_bytes,
                                                   uint32_t sbo_bytes, uint32_t swizzle_mode)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(swizzle_mode & 7u) << 61;
    return d;
}

// ---------------------------------------------------------------- Philox4x32-10
// Counter-based generator of the stochastic-rounding variant: same inputs, same outputs on
// any thread, so the stream is a pure function of (seed, counter).  The ten round keys
// (key + r * Weyl constant, the published key schedule) depend on the seed only, so the host
// computes them once per call and the kernel reads them as constant-bank operands of the XORs;
// each round is then two 32 x 32 -> 64-bit multiplies and two three-input XORs.
struct PhiloxRoundKeys {
    uint32_t k0[10], k1[10];
};

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              const PhiloxRoundKeys& rk, uint32_t (&out)[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = static_cast<uint64_t>(0xD2511F53u) * c0;
        const uint64_t p1 = static_cast<uint64_t>(0xCD9E8D57u) * c2;
        const uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c1 ^ rk.k0[r];
        const uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c3 ^ rk.k1[r];
        c0 = n0; c1 = static_cast<uint32_t>(p1); c2 = n2; c3 = static_cast<uint32_t>(p0);
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// byte permute: byte i of the result is byte (selector nibble i) of the eight bytes {a, b}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t selector)
{
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(selector));
    return r;
}

// minimum of the two unsigned 16-bit halves
__device__ __forceinline__ uint32_t min_u16x2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("min.u16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

}  // namespace mxfp4

// ------------------------------------------------------------------ CTA pairs (cluster of 2)
namespace mxfp4 {

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}

__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Arrive (and add expected bytes) on a barrier given by its shared::cluster address.  These
// signals publish no ordinary memory writes of the arriving thread -- what they announce was
// produced by TMA (counted separately by complete_tx) or by tcgen05 operations the thread has
// already waited for -- so they are relaxed; a cluster-scope release costs about a thousand
// cycles per arrive, which is more than a whole K-step of MMAs.
__device__ __forceinline__ void mbar_arrive_expect_tx_cluster(uint32_t cluster_addr, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.relaxed.cluster.shared::cluster.b64 _, [%0], %1;"
                 ::"r"(cluster_addr), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr)
                 : "memory");
}

// 2-D tiled load whose completion is counted on a barrier that may live in the peer CTA of the
// pair (the data lands only in the executing CTA's shared memory).
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const void* tmap, uint32_t bar_cluster_addr,
                                                 int32_t x, int32_t y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar_cluster_addr),
        "r"(x), "r"(y)
        : "memory");
}

__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_result, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(smem_result)), "r"(ncols)
                 : "memory");
}

__device__ __forceinline__ void tmem_relinquish_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
                 : "memory");
}

// Arrive on the barrier at this shared-memory offset in every CTA of `cta_mask` once all
// tcgen05 operations issued so far by this thread have completed.
__device__ __forceinline__ void tcgen05_commit_pair(uint64_t* bar, uint16_t cta_mask)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(smem_u32(bar)), "h"(cta_mask)
        : "memory");
}

// Pair MMA, 256 x N x 64 (or x 32) across the two CTAs (each holds 128 rows of A and N/2 rows of B):
// D[tmem] (+)= A[smem] * B[smem]^T with E8M0 scales in TMEM.  A-collector hint: FILL keeps the A operand in the collector buffer for the
// next MMA, LASTUSE consumes the kept copy (two MMAs that share A read it from shared memory once).
// KIND 0: 4-bit operands (kind::mxf4, K = 64, two scales per row: scale_vec::2X);
// KIND 1: 8-bit operands (kind::mxf8f6f4, K = 32, one scale per row: scale_vec::1X).
#define MXFP4_PAIR_MMA(KIND_STR, HINT)                                                                  \
    asm volatile(                                                                                       \
        "{\n\t.reg .pred P;\n\t"                                                                       \
        "setp.ne.b32 P, %6, 0;\n\t"                                                                     \
        "tcgen05.mma.cta_group::2." KIND_STR ".collector::a::" HINT " "                                 \
        "[%0], %1, %2, %3, [%4], [%5], P;\n\t}"                                                         \
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem), "r"(accumulate) \
        : "memory")

template <int KIND, int LAST>
__device__ __forceinline__ void tcgen05_mma_mx_pair_collect(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                                            uint32_t idesc, uint32_t sfa_tmem,
                                                            uint32_t sfb_tmem, uint32_t accumulate)
{
    if (KIND == 0) {
        if (LAST) MXFP4_PAIR_MMA("kind::mxf4.block_scale.scale_vec::2X", "lastuse");
        else      MXFP4_PAIR_MMA("kind::mxf4.block_scale.scale_vec::2X", "fill");
    } else {
        if (LAST) MXFP4_PAIR_MMA("kind::mxf8f6f4.block_scale.scale_vec::1X", "lastuse");
        else      MXFP4_PAIR_MMA("kind::mxf8f6f4.block_scale.scale_vec::1X", "fill");
    }
}
#undef MXFP4_PAIR_MMA

}  // namespace mxfp4
