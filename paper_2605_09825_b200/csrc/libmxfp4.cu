// C ABI of the library (see include/mxfp4.h).  Single translation unit: the kernels live in
// the headers included below.  Host code here only validates arguments, builds TMA tensor
// maps and launches; every step of the path runs in the kernels.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <mutex>

#include "../../include/mxfp4.h"
#include "ptx_sm100.cuh"
#include "tma_host.cuh"
#include "quantize_kernel.cuh"
#include "quantize_dual_kernel.cuh"
#include "quantize_fp8_kernel.cuh"
#include "gemm_pair_kernel.cuh"
#include "mma_rate_probe.cuh"

namespace mxfp4 {

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

constexpr int kMaxDevices = 64;      // size of the per-device tables below

struct DeviceInfo {
    int sm_count = 0;
    int cc_major = 0;
    bool ok = false;
};

// Per-device set-up that runs once however many host threads reach it at the same time: the
// first caller on a device runs `f` (which returns a status code), the others wait for it, and
// everybody gets that status.  One instance per table (device properties, a kernel's
// shared-memory attribute, the copy streams of the host-buffer call, ...).
struct PerDeviceOnce {
    std::once_flag flag[kMaxDevices];
    int status[kMaxDevices] = {};
    template <class F>
    int run(int dev, F&& f)
    {
        std::call_once(flag[dev], [&] { status[dev] = f(); });
        return status[dev];
    }
};

// Ordinal of the current device, or -1 if it cannot be had or lies beyond the tables.
static int current_device()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}

static const DeviceInfo& device_info()
{
    static DeviceInfo info[kMaxDevices];
    static PerDeviceOnce once;
    static const DeviceInfo none;
    const int dev = current_device();
    if (dev < 0) return none;
    once.run(dev, [&] {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) == cudaSuccess) {
            info[dev].sm_count = prop.multiProcessorCount;
            info[dev].cc_major = prop.major;
            info[dev].ok = true;
        }
        return 0;
    });
    return info[dev];
}

// Raises a kernel's dynamic shared-memory limit on the current device, once per device.
template <class Kernel>
static int ensure_smem_attribute(PerDeviceOnce& once, Kernel kernel, size_t smem)
{
    const int dev = current_device();
    if (dev < 0) return MXFP4_ERR_CUDA;
    return once.run(dev, [&] {
        return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) ==
                       cudaSuccess
                   ? MXFP4_OK : MXFP4_ERR_CUDA;
    });
}

// Host copy of the counter-based generator, used only for the 32-bit sign mask of the
// randomized rotation (counter (0,0,0,1), key = seed).
static uint32_t host_sign_mask(uint64_t seed)
{
    uint32_t c[4] = {0, 0, 0, 1};
    uint32_t k0 = static_cast<uint32_t>(seed), k1 = static_cast<uint32_t>(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = 0xD2511F53ull * c[0], p1 = 0xCD9E8D57ull * c[2];
        const uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c[1] ^ k0;
        const uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c[3] ^ k1;
        c[0] = n0; c[1] = static_cast<uint32_t>(p1); c[2] = n2; c[3] = static_cast<uint32_t>(p0);
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return c[0];
}

template <int AXIS0, int AXIS1, int HMODE, int SR, bool PLAIN>
static int launch_quantize_as(const QuantJob& j0, const QuantJob& j1, int grid, cudaStream_t stream)
{
    const size_t smem = sizeof(QuantSmem) + 1024;
    static PerDeviceOnce once;               // the attribute is per device
    const int rc = ensure_smem_attribute(once, quantize_kernel<AXIS0, AXIS1, HMODE, SR, PLAIN>, smem);
    if (rc != MXFP4_OK) return rc;
    QuantJobs jobs;
    jobs.j[0] = j0;
    jobs.j[1] = j1;
    return launch_kernel_pdl(quantize_kernel<AXIS0, AXIS1, HMODE, SR, PLAIN>, grid, kQThreads, smem, stream, jobs) ==
                   cudaSuccess
               ? MXFP4_OK : MXFP4_ERR_CUDA;
}

template <int AXIS0, int AXIS1, int HMODE, int SR>
static int launch_quantize(const QuantJob& j0, const QuantJob& j1, int grid, cudaStream_t stream)
{
    // what the fused passes use (tiled scales, 1 x 32 blocks, in both jobs) has an instantiation of its own
    const bool plain0 = j0.p.scale_layout == MXFP4_SCALES_TILED && !j0.p.block2d;
    const bool plain1 = j1.tiles == 0 || (j1.p.scale_layout == MXFP4_SCALES_TILED && !j1.p.block2d);
    if (plain0 && plain1) return launch_quantize_as<AXIS0, AXIS1, HMODE, SR, true>(j0, j1, grid, stream);
    return launch_quantize_as<AXIS0, AXIS1, HMODE, SR, false>(j0, j1, grid, stream);
}

template <int AXIS0, int AXIS1>
static int dispatch_quantize(int hmode, int sr, const QuantJob& j0, const QuantJob& j1, int grid,
                             cudaStream_t st)
{
    switch (hmode * 2 + sr) {
        case 0: return launch_quantize<AXIS0, AXIS1, 0, 0>(j0, j1, grid, st);
        case 1: return launch_quantize<AXIS0, AXIS1, 0, 1>(j0, j1, grid, st);
        case 2: return launch_quantize<AXIS0, AXIS1, 1, 0>(j0, j1, grid, st);
        case 3: return launch_quantize<AXIS0, AXIS1, 1, 1>(j0, j1, grid, st);
        case 4: return launch_quantize<AXIS0, AXIS1, 2, 0>(j0, j1, grid, st);
        case 5: return launch_quantize<AXIS0, AXIS1, 2, 1>(j0, j1, grid, st);
        case 6: return launch_quantize<AXIS0, AXIS1, 3, 0>(j0, j1, grid, st);
        case 7: return launch_quantize<AXIS0, AXIS1, 3, 1>(j0, j1, grid, st);
        case 8: return launch_quantize<AXIS0, AXIS1, 4, 0>(j0, j1, grid, st);
        default: return launch_quantize<AXIS0, AXIS1, 4, 1>(j0, j1, grid, st);
    }
}

static void fill_quant_params(QuantParams* pp, int64_t outer, int64_t K, int hadamard_mode, uint64_t seed,
                              uint32_t operand_tag, void* scales, int scale_layout, int block2d)
{
    QuantParams& p = *pp;
    p.scales = static_cast<uint8_t*>(scales);
    p.outer = outer;
    p.K = K;
    p.nt = K / 32;
    p.tiles_o = static_cast<int32_t>((outer + kQTileO - 1) / kQTileO);
    p.tiles_k = static_cast<int32_t>((K + kQTileK - 1) / kQTileK);
    for (int r = 0; r < 10; ++r) {          // key schedule of Philox4x32-10: key + r * Weyl constant
        p.rk.k0[r] = static_cast<uint32_t>(seed) + static_cast<uint32_t>(r) * 0x9E3779B9u;
        p.rk.k1[r] = static_cast<uint32_t>(seed >> 32) + static_cast<uint32_t>(r) * 0xBB67AE85u;
    }
    p.tag = operand_tag;
    p.sign_mask = 0u;
    if (hadamard_mode == MXFP4_HADAMARD_RAND) p.sign_mask = host_sign_mask(seed);
    if (hadamard_mode == MXFP4_HADAMARD_RAND16) {
        const uint32_t m16 = host_sign_mask(seed) & 0xFFFFu;   // same 16 signs for both halves
        p.sign_mask = m16 | (m16 << 16);
    }
    for (int i = 0; i < 16; ++i)
        p.signs.pair[i] = (((p.sign_mask >> (2 * i)) & 1u) << 15) | (((p.sign_mask >> (2 * i + 1)) & 1u) << 31);
    for (int k = 0; k < 32; ++k) p.signs.word[k] = ((p.sign_mask >> k) & 1u) ? 0x80008000u : 0u;
    p.scale_layout = scale_layout;
    p.block2d = block2d;
}

// Size limits of the kernels' 32-bit tile arithmetic, checked on the host before anything else is
// done with a shape: a quantizer walks at most 2^30 source tiles of 128 x 128, a GEMM at most 2^30
// output tiles of 256 x 384 and fewer than 2^31 (output tile, K-step of 256 elements) pairs.
static bool quant_tiles_fit(int64_t rows, int64_t cols)
{
    return ((rows + 127) / 128) * ((cols + 127) / 128) <= 0x3FFFFFFF;
}

static bool gemm_tiles_fit(int64_t M, int64_t N, int64_t K)
{
    const int64_t tiles = ((M + kPTileM - 1) / kPTileM) * ((N + kPTileN - 1) / kPTileN);
    if (tiles > 0x3FFFFFFF) return false;
    const int64_t k_steps = (K + 127) / 128;              // the 8-bit kernel's K-step; the 4-bit one's is 256
    return tiles <= 0x7FFFFFFF / k_steps;
}

// Validates one tensor's arguments and fills its job (tensor maps + parameters).
static int build_quant_job(const void* src_bf16, int64_t rows, int64_t cols, int64_t ld_src, int axis,
                           int hadamard_mode, int rounding, uint64_t seed, uint32_t operand_tag,
                           void* codes, void* scales, int scale_layout, QuantJob* job, int block2d = 0,
                           int fp8 = 0)
{
    if (!src_bf16 || !codes || !scales) return MXFP4_ERR_NULL;
    if (axis != 0 && axis != 1) return MXFP4_ERR_ENUM;
    if (hadamard_mode < 0 || hadamard_mode > 4 || rounding < 0 || rounding > 1) return MXFP4_ERR_ENUM;
    if (scale_layout != 0 && scale_layout != 1) return MXFP4_ERR_ENUM;
    if (rows <= 0 || cols <= 0 || ld_src < cols) return MXFP4_ERR_SHAPE;
    const int64_t outer = axis ? rows : cols;
    const int64_t K = axis ? cols : rows;
    if (K % 32 != 0) return MXFP4_ERR_SHAPE;
    if (rows > 0x7FFFFFFF || cols > 0x7FFFFFFF || !quant_tiles_fit(rows, cols)) return MXFP4_ERR_SHAPE;
    if (!aligned16(src_bf16) || !aligned16(codes) || !aligned16(scales)) return MXFP4_ERR_ALIGN;
    if (ld_src % 8 != 0) return MXFP4_ERR_ALIGN;
    const DeviceInfo& dev = device_info();
    if (!dev.ok) return MXFP4_ERR_CUDA;
    if (dev.cc_major != 10) return MXFP4_ERR_DEVICE;

    const bool ok_src =
        axis == 1 ? make_tmap_2d(&job->tm_src, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, src_bf16, rows, cols,
                                 ld_src * 2, 128, 64, CU_TENSOR_MAP_SWIZZLE_128B)
                  : make_tmap_2d(&job->tm_src, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, src_bf16, rows, cols,
                                 ld_src * 2, 128, 128, CU_TENSOR_MAP_SWIZZLE_NONE);
    const bool ok_codes =
        fp8 ? make_tmap_2d(&job->tm_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, codes, outer, K, K, 128, 128,
                           CU_TENSOR_MAP_SWIZZLE_128B)
            : make_tmap_2d(&job->tm_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, codes, outer, K / 2, K / 2, 128, 64,
                           CU_TENSOR_MAP_SWIZZLE_64B);
    if (!ok_src || !ok_codes) return MXFP4_ERR_CUDA;

    QuantParams& p = job->p;
    fill_quant_params(&p, outer, K, hadamard_mode, seed, operand_tag, scales, scale_layout, block2d);
    const int64_t total = static_cast<int64_t>(p.tiles_o) * p.tiles_k;
    if (total > 0x3FFFFFFF) return MXFP4_ERR_SHAPE;
    job->tiles = static_cast<int32_t>(total);
    return MXFP4_OK;
}

// One launch for one or two jobs (axis1 is ignored when j1 is empty).
static int launch_quant_jobs(const QuantJob& j0, const QuantJob& j1, int axis0, int axis1, int hmode, int sr,
                             cudaStream_t st)
{
    const DeviceInfo& dev = device_info();
    const int64_t total = static_cast<int64_t>(j0.tiles) + j1.tiles;
    const int grid = static_cast<int>(total < dev.sm_count ? total : dev.sm_count);
    if (j1.tiles == 0) axis1 = axis0;
    if (axis0 == 1 && axis1 == 1) return dispatch_quantize<1, 1>(hmode, sr, j0, j1, grid, st);
    if (axis0 == 1 && axis1 == 0) return dispatch_quantize<1, 0>(hmode, sr, j0, j1, grid, st);
    if (axis0 == 0 && axis1 == 0) return dispatch_quantize<0, 0>(hmode, sr, j0, j1, grid, st);
    return MXFP4_ERR_ENUM;   // (0, 1) is never asked for: callers order row-wise first
}

template <int AXIS0, int AXIS1>
static int launch_quantize_fp8(const QuantJob& j0, const QuantJob& j1, int grid, cudaStream_t stream)
{
    const size_t smem = sizeof(QuantFp8Smem) + 1024;
    static PerDeviceOnce once;               // the attribute is per device
    const int rc = ensure_smem_attribute(once, quantize_fp8_kernel<AXIS0, AXIS1>, smem);
    if (rc != MXFP4_OK) return rc;
    QuantJobs jobs;
    jobs.j[0] = j0;
    jobs.j[1] = j1;
    return launch_kernel_pdl(quantize_fp8_kernel<AXIS0, AXIS1>, grid, kQThreads, smem, stream, jobs) == cudaSuccess
               ? MXFP4_OK : MXFP4_ERR_CUDA;
}

static int launch_quant_jobs_fp8(const QuantJob& j0, const QuantJob& j1, int axis0, int axis1, cudaStream_t st)
{
    const DeviceInfo& dev = device_info();
    const int64_t total = static_cast<int64_t>(j0.tiles) + j1.tiles;
    const int grid = static_cast<int>(total < dev.sm_count ? total : dev.sm_count);
    if (j1.tiles == 0) axis1 = axis0;
    if (axis0 == 1 && axis1 == 1) return launch_quantize_fp8<1, 1>(j0, j1, grid, st);
    if (axis0 == 1 && axis1 == 0) return launch_quantize_fp8<1, 0>(j0, j1, grid, st);
    if (axis0 == 0 && axis1 == 0) return launch_quantize_fp8<0, 0>(j0, j1, grid, st);
    return MXFP4_ERR_ENUM;
}

template <int HMODE, int SR, bool PLAIN>
static int launch_quantize_dual_as(const QuantDualJob& job, int grid, cudaStream_t stream)
{
    const size_t smem = sizeof(QuantDualSmem) + 1024;
    static PerDeviceOnce once;               // the attribute is per device
    const int rc = ensure_smem_attribute(once, quantize_dual_kernel<HMODE, SR, PLAIN>, smem);
    if (rc != MXFP4_OK) return rc;
    return launch_kernel_pdl(quantize_dual_kernel<HMODE, SR, PLAIN>, grid, kQThreads, smem, stream, job) == cudaSuccess
               ? MXFP4_OK : MXFP4_ERR_CUDA;
}

template <int HMODE, int SR>
static int launch_quantize_dual(const QuantDualJob& job, int grid, cudaStream_t stream)
{
    // the layer-level path (tiled scales, 1 x 32 blocks) has an instantiation of its own
    if (!QuantDualShape<HMODE, SR>::kFirstForm && job.pr.scale_layout == MXFP4_SCALES_TILED && !job.pr.block2d)
        return launch_quantize_dual_as<HMODE, SR, true>(job, grid, stream);
    return launch_quantize_dual_as<HMODE, SR, false>(job, grid, stream);
}

static size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Self-test of the bounded-wait discipline: one warp waits on a barrier that nothing will ever
// complete, with a spin limit of a few hundred attempts.  The wait gives up, records the
// timeout status and the kernel returns normally.
__global__ void selftest_wait_timeout_kernel()
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&bar, 1);
        fence_barrier_init();
    }
    __syncthreads();
    mbar_wait(&bar, 0, &abort_flag, 256u);
}

// Self-test of the bounds discipline: the checker is handed an address one element past a
// shared array.  It refuses (the store never happens) and records the status.
__global__ void selftest_bounds_kernel()
{
    __shared__ uint32_t buf[8];
    uint32_t* past = buf + 8;
    if (bounds_ok(past, sizeof(uint32_t), buf, sizeof(buf))) *past = 1u;
}

}  // namespace mxfp4

using namespace mxfp4;

template <int KIND>
static int gemm_checked(const void* a_codes, const void* a_scales, const void* b_codes, const void* b_scales,
                        int64_t M, int64_t N, int64_t K, float alpha, void* out, int out_dtype, int64_t ld_out,
                        void* stream)
{
    if (!a_codes || !a_scales || !b_codes || !b_scales || !out) return MXFP4_ERR_NULL;
    if (out_dtype != MXFP4_OUT_BF16 && out_dtype != MXFP4_OUT_FP32) return MXFP4_ERR_ENUM;
    if (M <= 0 || N <= 0 || K <= 0 || K % 32 != 0 || ld_out < N) return MXFP4_ERR_SHAPE;
    if (M > 0x7FFFFFFF || N > 0x7FFFFFFF || K > 0x7FFFFFFF || !gemm_tiles_fit(M, N, K)) return MXFP4_ERR_SHAPE;
    if (!aligned16(a_codes) || !aligned16(a_scales) || !aligned16(b_codes) || !aligned16(b_scales) ||
        !aligned16(out))
        return MXFP4_ERR_ALIGN;
    const int64_t esz = out_dtype == MXFP4_OUT_BF16 ? 2 : 4;
    if ((ld_out * esz) % 16 != 0) return MXFP4_ERR_ALIGN;
    const DeviceInfo& dev = device_info();
    if (!dev.ok) return MXFP4_ERR_CUDA;
    if (dev.cc_major != 10) return MXFP4_ERR_DEVICE;
    return launch_gemm_pair<KIND>(a_codes, a_scales, b_codes, b_scales, M, N, K, alpha, out, out_dtype, ld_out,
                                  dev.sm_count, static_cast<cudaStream_t>(stream));
}

extern "C" {

int mxfp4_version(void) { return 106; }   // 1.6: shared-space accesses in the quantizers, size limits checked on the host

const char* mxfp4_status_string(int status)
{
    switch (status) {
        case MXFP4_OK: return "ok";
        case MXFP4_ERR_NULL: return "null pointer";
        case MXFP4_ERR_SHAPE: return "bad shape";
        case MXFP4_ERR_ALIGN: return "bad alignment";
        case MXFP4_ERR_ENUM: return "bad enum value";
        case MXFP4_ERR_WORKSPACE: return "workspace missing or too small";
        case MXFP4_ERR_CUDA: return "CUDA call failed";
        case MXFP4_ERR_TIMEOUT: return "device-side wait timed out";
        case MXFP4_ERR_DEVICE: return "not an sm_100 device";
        case MXFP4_ERR_STATIC_LIMIT: return "problem needs more scratch than the built-in array holds";
        case MXFP4_ERR_BOUNDS: return "a kernel computed an address outside its buffer (debug build)";
        default: return "unknown status";
    }
}

size_t mxfp4_codes_bytes(int64_t outer, int64_t K)
{
    if (outer <= 0 || K <= 0 || K % 32 != 0) return 0;
    return static_cast<size_t>(outer) * static_cast<size_t>(K / 2);
}

size_t mxfp4_scales_bytes(int64_t outer, int64_t K, int scale_layout)
{
    if (outer <= 0 || K <= 0 || K % 32 != 0) return 0;
    if (scale_layout == MXFP4_SCALES_CANONICAL)
        return static_cast<size_t>(outer) * static_cast<size_t>(K / 32);
    if (scale_layout == MXFP4_SCALES_TILED)
        return static_cast<size_t>((outer + 127) / 128) * static_cast<size_t>((K + 127) / 128) * 512;
    return 0;
}

int mxfp4_quantize(const void* src_bf16, int64_t rows, int64_t cols, int64_t ld_src, int axis,
                   int hadamard_mode, int rounding, uint64_t seed, uint32_t operand_tag,
                   void* codes, void* scales, int scale_layout, void* stream)
{
    QuantJob j0, j1;
    const int rc = build_quant_job(src_bf16, rows, cols, ld_src, axis, hadamard_mode, rounding, seed,
                                   operand_tag, codes, scales, scale_layout, &j0);
    if (rc != MXFP4_OK) return rc;
    memset(&j1, 0, sizeof(j1));
    return launch_quant_jobs(j0, j1, axis, axis, hadamard_mode, rounding, static_cast<cudaStream_t>(stream));
}

int mxfp4_quantize_2d(const void* src_bf16, int64_t rows, int64_t cols, int64_t ld_src, int axis,
                      int hadamard_mode, int rounding, uint64_t seed, uint32_t operand_tag,
                      void* codes, void* scales, int scale_layout, void* stream)
{
    QuantJob j0, j1;
    const int rc = build_quant_job(src_bf16, rows, cols, ld_src, axis, hadamard_mode, rounding, seed,
                                   operand_tag, codes, scales, scale_layout, &j0, 1);
    if (rc != MXFP4_OK) return rc;
    memset(&j1, 0, sizeof(j1));
    return launch_quant_jobs(j0, j1, axis, axis, hadamard_mode, rounding, static_cast<cudaStream_t>(stream));
}

int mxfp4_quantize_dual(const void* src_bf16, int64_t rows, int64_t cols, int64_t ld_src, int hadamard_mode,
                        int rounding, uint64_t seed, uint32_t tag_rowwise, uint32_t tag_colwise,
                        int block_shape, void* codes_rowwise, void* scales_rowwise, void* codes_colwise,
                        void* scales_colwise, int scale_layout, void* stream)
{
    if (!src_bf16 || !codes_rowwise || !scales_rowwise || !codes_colwise || !scales_colwise) return MXFP4_ERR_NULL;
    if (hadamard_mode < 0 || hadamard_mode > 4 || rounding < 0 || rounding > 1) return MXFP4_ERR_ENUM;
    if (scale_layout != 0 && scale_layout != 1) return MXFP4_ERR_ENUM;
    if (block_shape != MXFP4_BLOCK_1X32 && block_shape != MXFP4_BLOCK_32X32) return MXFP4_ERR_ENUM;
    if (rows <= 0 || cols <= 0 || ld_src < cols) return MXFP4_ERR_SHAPE;
    if (rows % 32 != 0 || cols % 32 != 0) return MXFP4_ERR_SHAPE;      // both axes are reduction axes here
    if (rows > 0x7FFFFFFF || cols > 0x7FFFFFFF || !quant_tiles_fit(rows, cols)) return MXFP4_ERR_SHAPE;
    if (!aligned16(src_bf16) || !aligned16(codes_rowwise) || !aligned16(scales_rowwise) ||
        !aligned16(codes_colwise) || !aligned16(scales_colwise))
        return MXFP4_ERR_ALIGN;
    if (ld_src % 8 != 0) return MXFP4_ERR_ALIGN;
    const DeviceInfo& dev = device_info();
    if (!dev.ok) return MXFP4_ERR_CUDA;
    if (dev.cc_major != 10) return MXFP4_ERR_DEVICE;

    QuantDualJob job;
    const bool ok = make_tmap_2d(&job.tm_src, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, src_bf16, rows, cols, ld_src * 2,
                                 128, 64, CU_TENSOR_MAP_SWIZZLE_128B) &&
                    make_tmap_2d(&job.tm_codes_row, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, codes_rowwise, rows, cols / 2,
                                 cols / 2, 128, 64, CU_TENSOR_MAP_SWIZZLE_64B) &&
                    make_tmap_2d(&job.tm_codes_col, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, codes_colwise, cols, rows / 2,
                                 rows / 2, 128, 64, CU_TENSOR_MAP_SWIZZLE_64B);
    if (!ok) return MXFP4_ERR_CUDA;
    const int b2d = block_shape == MXFP4_BLOCK_32X32;
    fill_quant_params(&job.pr, rows, cols, hadamard_mode, seed, tag_rowwise, scales_rowwise, scale_layout, b2d);
    fill_quant_params(&job.pc, cols, rows, hadamard_mode, seed, tag_colwise, scales_colwise, scale_layout, b2d);
    job.tiles_r = job.pr.tiles_o;
    job.tiles_c = job.pr.tiles_k;
    const int64_t total = static_cast<int64_t>(job.tiles_r) * job.tiles_c;
    if (total > 0x3FFFFFFF) return MXFP4_ERR_SHAPE;
    const int grid = static_cast<int>(total < dev.sm_count ? total : dev.sm_count);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    switch (hadamard_mode * 2 + rounding) {
        case 0: return launch_quantize_dual<0, 0>(job, grid, st);
        case 1: return launch_quantize_dual<0, 1>(job, grid, st);
        case 2: return launch_quantize_dual<1, 0>(job, grid, st);
        case 3: return launch_quantize_dual<1, 1>(job, grid, st);
        case 4: return launch_quantize_dual<2, 0>(job, grid, st);
        case 5: return launch_quantize_dual<2, 1>(job, grid, st);
        case 6: return launch_quantize_dual<3, 0>(job, grid, st);
        case 7: return launch_quantize_dual<3, 1>(job, grid, st);
        case 8: return launch_quantize_dual<4, 0>(job, grid, st);
        default: return launch_quantize_dual<4, 1>(job, grid, st);
    }
}

int mxfp4_quantize_pair(const mxfp4_quant_desc* a, const mxfp4_quant_desc* b, int hadamard_mode,
                        int rounding, uint64_t seed, int scale_layout, void* stream)
{
    if (!a || !b) return MXFP4_ERR_NULL;
    if (a->axis == MXFP4_AXIS_ROWS && b->axis == MXFP4_AXIS_COLS) return MXFP4_ERR_ENUM;
    QuantJob ja, jb;
    int rc = build_quant_job(a->src_bf16, a->rows, a->cols, a->ld_src, a->axis, hadamard_mode, rounding, seed,
                             a->operand_tag, a->codes, a->scales, scale_layout, &ja);
    if (rc != MXFP4_OK) return rc;
    rc = build_quant_job(b->src_bf16, b->rows, b->cols, b->ld_src, b->axis, hadamard_mode, rounding, seed,
                         b->operand_tag, b->codes, b->scales, scale_layout, &jb);
    if (rc != MXFP4_OK) return rc;
    return launch_quant_jobs(ja, jb, a->axis, b->axis, hadamard_mode, rounding, static_cast<cudaStream_t>(stream));
}

int mxfp4_gemm(const void* a_codes, const void* a_scales, const void* b_codes,
               const void* b_scales, int64_t M, int64_t N, int64_t K, float alpha, void* out,
               int out_dtype, int64_t ld_out, void* workspace, size_t workspace_bytes,
               void* stream)
{
    (void)workspace;
    (void)workspace_bytes;
    return gemm_checked<0>(a_codes, a_scales, b_codes, b_scales, M, N, K, alpha, out, out_dtype, ld_out, stream);
}

int mxfp4_gemm_fp8(const void* a_codes, const void* a_scales, const void* b_codes, const void* b_scales,
                   int64_t M, int64_t N, int64_t K, float alpha, void* out, int out_dtype, int64_t ld_out,
                   void* stream)
{
    return gemm_checked<1>(a_codes, a_scales, b_codes, b_scales, M, N, K, alpha, out, out_dtype, ld_out, stream);
}

int mxfp4_quantize_fp8(const void* src_bf16, int64_t rows, int64_t cols, int64_t ld_src, int axis, void* codes,
                       void* scales, int scale_layout, void* stream)
{
    QuantJob j0, j1;
    const int rc = build_quant_job(src_bf16, rows, cols, ld_src, axis, MXFP4_HADAMARD_NONE, MXFP4_ROUND_RNE, 0, 0u,
                                   codes, scales, scale_layout, &j0, 0, 1);
    if (rc != MXFP4_OK) return rc;
    memset(&j1, 0, sizeof(j1));
    return launch_quant_jobs_fp8(j0, j1, axis, axis, static_cast<cudaStream_t>(stream));
}

// Workspace layout of a fused pass: [A codes][A scales][B codes][B scales], each region
// rounded up to 256 bytes.
static void linear_dims(int pass, int64_t T, int64_t in_f, int64_t out_f, int64_t* M, int64_t* N,
                        int64_t* K)
{
    if (pass == MXFP4_PASS_FPROP) { *M = T; *N = out_f; *K = in_f; }
    else if (pass == MXFP4_PASS_DGRAD) { *M = T; *N = in_f; *K = out_f; }
    else { *M = out_f; *N = in_f; *K = T; }
}

size_t mxfp4_linear_workspace_bytes(int64_t T, int64_t in_features, int64_t out_features, int pass)
{
    if (pass < 0 || pass > 2 || T <= 0 || in_features <= 0 || out_features <= 0) return 0;
    int64_t M, N, K;
    linear_dims(pass, T, in_features, out_features, &M, &N, &K);
    if (K % 32 != 0) return 0;
    return round_up(mxfp4_codes_bytes(M, K), 256) + round_up(mxfp4_scales_bytes(M, K, 1), 256) +
           round_up(mxfp4_codes_bytes(N, K), 256) + round_up(mxfp4_scales_bytes(N, K, 1), 256);
}

static size_t pass_workspace_bytes(int64_t T, int64_t in_features, int64_t out_features, int pass, int precision)
{
    if (pass < 0 || pass > 2 || T <= 0 || in_features <= 0 || out_features <= 0) return 0;
    if (precision < MXFP4_PRECISION_MXFP4 || precision > MXFP4_PRECISION_MXFP4_32X32) return 0;
    int64_t M, N, K;
    linear_dims(pass, T, in_features, out_features, &M, &N, &K);
    if (K % 32 != 0) return 0;
    const size_t mul = precision == MXFP4_PRECISION_MXFP8 ? 2 : 1;     // one byte per element instead of half
    return round_up(mul * mxfp4_codes_bytes(M, K), 256) + round_up(mxfp4_scales_bytes(M, K, 1), 256) +
           round_up(mul * mxfp4_codes_bytes(N, K), 256) + round_up(mxfp4_scales_bytes(N, K, 1), 256);
}

static int linear_pass(int pass, const void* a_src, const void* b_src, void* out, int64_t T,
                       int64_t in_f, int64_t out_f, int hmode, int rounding, uint64_t seed,
                       int out_dtype, void* workspace, size_t workspace_bytes, void* stream,
                       int precision = MXFP4_PRECISION_MXFP4, bool validate_only = false)
{
    const bool fp8 = precision == MXFP4_PRECISION_MXFP8;
    const int b2d = precision == MXFP4_PRECISION_MXFP4_32X32 ? 1 : 0;    // Appendix D's 32 x 32 blocks
    const size_t cmul = fp8 ? 2 : 1;
    if (!a_src || !b_src || !out) return MXFP4_ERR_NULL;
    if (T <= 0 || in_f <= 0 || out_f <= 0) return MXFP4_ERR_SHAPE;
    if (hmode < 0 || hmode > 4 || rounding < 0 || rounding > 1) return MXFP4_ERR_ENUM;
    int64_t M, N, K;
    linear_dims(pass, T, in_f, out_f, &M, &N, &K);
    if (K % 32 != 0 || in_f % 8 != 0 || out_f % 8 != 0) return MXFP4_ERR_SHAPE;
    // everything the GEMM would reject is checked here, before the quantize launch
    if (out_dtype != MXFP4_OUT_BF16 && out_dtype != MXFP4_OUT_FP32) return MXFP4_ERR_ENUM;
    if (M > 0x7FFFFFFF || N > 0x7FFFFFFF || K > 0x7FFFFFFF) return MXFP4_ERR_SHAPE;
    if (!gemm_tiles_fit(M, N, K) || !quant_tiles_fit(M, K) || !quant_tiles_fit(N, K)) return MXFP4_ERR_SHAPE;
    const size_t need = pass_workspace_bytes(T, in_f, out_f, pass, precision);
    if (!workspace || workspace_bytes < need) return MXFP4_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return MXFP4_ERR_ALIGN;
    if (!aligned16(a_src) || !aligned16(b_src) || !aligned16(out)) return MXFP4_ERR_ALIGN;
    if (validate_only) return MXFP4_OK;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    uint8_t* a_codes = ws;
    uint8_t* a_scales = a_codes + round_up(cmul * mxfp4_codes_bytes(M, K), 256);
    uint8_t* b_codes = a_scales + round_up(mxfp4_scales_bytes(M, K, 1), 256);
    uint8_t* b_scales = b_codes + round_up(cmul * mxfp4_codes_bytes(N, K), 256);

    // (rows, cols, axis) of each source in its own row-major shape
    int64_t ar, ac, br, bc;
    int a_axis, b_axis;
    if (pass == MXFP4_PASS_FPROP) {          // A = X [T x in] row-wise, B = W [out x in] row-wise
        ar = T; ac = in_f; a_axis = 1; br = out_f; bc = in_f; b_axis = 1;
    } else if (pass == MXFP4_PASS_DGRAD) {   // A = dY [T x out] row-wise, B = W [out x in] column-wise
        ar = T; ac = out_f; a_axis = 1; br = out_f; bc = in_f; b_axis = 0;
    } else {                                 // A = dY [T x out] column-wise, B = X [T x in] column-wise
        ar = T; ac = out_f; a_axis = 0; br = T; bc = in_f; b_axis = 0;
    }
    // both operands through one quantize launch
    QuantJob ja, jb;
    if (fp8) hmode = MXFP4_HADAMARD_NONE, rounding = MXFP4_ROUND_RNE;    // the stabilisers belong to the 4-bit GEMMs
    int rc = build_quant_job(a_src, ar, ac, ac, a_axis, hmode, rounding, seed, 0u, a_codes, a_scales,
                             MXFP4_SCALES_TILED, &ja, b2d, fp8);
    if (rc != MXFP4_OK) return rc;
    rc = build_quant_job(b_src, br, bc, bc, b_axis, hmode, rounding, seed, 1u, b_codes, b_scales,
                         MXFP4_SCALES_TILED, &jb, b2d, fp8);
    if (rc != MXFP4_OK) return rc;
    rc = fp8 ? launch_quant_jobs_fp8(ja, jb, a_axis, b_axis, static_cast<cudaStream_t>(stream))
             : launch_quant_jobs(ja, jb, a_axis, b_axis, hmode, rounding, static_cast<cudaStream_t>(stream));
    if (rc != MXFP4_OK) return rc;
    if (fp8) return mxfp4_gemm_fp8(a_codes, a_scales, b_codes, b_scales, M, N, K, 1.0f, out, out_dtype, N, stream);
    // H * H^T = n * I for the +-1 matrix of order n: undo it exactly in the epilogue
    const float alpha = hmode == MXFP4_HADAMARD_NONE ? 1.0f : (hmode <= MXFP4_HADAMARD_RAND ? 0.03125f : 0.0625f);
    return mxfp4_gemm(a_codes, a_scales, b_codes, b_scales, M, N, K, alpha, out, out_dtype, N,
                      nullptr, 0, stream);
}

int mxfp4_linear_fprop(const void* X, const void* W, void* Y, int64_t T, int64_t in_features,
                       int64_t out_features, int hadamard_mode, int rounding, uint64_t seed,
                       int out_dtype, void* workspace, size_t workspace_bytes, void* stream)
{
    return linear_pass(MXFP4_PASS_FPROP, X, W, Y, T, in_features, out_features, hadamard_mode,
                       rounding, seed, out_dtype, workspace, workspace_bytes, stream);
}

int mxfp4_linear_dgrad(const void* dY, const void* W, void* dX, int64_t T, int64_t in_features,
                       int64_t out_features, int hadamard_mode, int rounding, uint64_t seed,
                       int out_dtype, void* workspace, size_t workspace_bytes, void* stream)
{
    return linear_pass(MXFP4_PASS_DGRAD, dY, W, dX, T, in_features, out_features, hadamard_mode,
                       rounding, seed, out_dtype, workspace, workspace_bytes, stream);
}

int mxfp4_linear_wgrad(const void* dY, const void* X, void* dW, int64_t T, int64_t in_features,
                       int64_t out_features, int hadamard_mode, int rounding, uint64_t seed,
                       int out_dtype, void* workspace, size_t workspace_bytes, void* stream)
{
    return linear_pass(MXFP4_PASS_WGRAD, dY, X, dW, T, in_features, out_features, hadamard_mode,
                       rounding, seed, out_dtype, workspace, workspace_bytes, stream);
}

size_t mxfp4_linear_pass_workspace_bytes(int64_t T, int64_t in_features, int64_t out_features, int pass,
                                         int precision)
{
    return pass_workspace_bytes(T, in_features, out_features, pass, precision);
}

int mxfp4_linear_pass(int pass, int precision, const void* a, const void* b, void* out, int64_t T,
                      int64_t in_features, int64_t out_features, int hadamard_mode, int rounding, uint64_t seed,
                      int out_dtype, void* workspace, size_t workspace_bytes, void* stream)
{
    if (pass < 0 || pass > 2) return MXFP4_ERR_ENUM;
    if (precision < MXFP4_PRECISION_MXFP4 || precision > MXFP4_PRECISION_MXFP4_32X32) return MXFP4_ERR_ENUM;
    return linear_pass(pass, a, b, out, T, in_features, out_features, hadamard_mode, rounding, seed, out_dtype,
                       workspace, workspace_bytes, stream, precision);
}

// Operand buffer = [codes][scales], each rounded up to 256 bytes.
static size_t operand_bytes(int64_t outer, int64_t K)
{
    return round_up(mxfp4_codes_bytes(outer, K), 256) + round_up(mxfp4_scales_bytes(outer, K, 1), 256);
}

size_t mxfp4_linear_layer_bytes(int64_t T, int64_t in_features, int64_t out_features, int which)
{
    if (T <= 0 || in_features <= 0 || out_features <= 0) return 0;
    if (T % 32 != 0 || in_features % 32 != 0 || out_features % 32 != 0) return 0;
    switch (which) {
        case MXFP4_LAYER_SAVED:      // X^T [in x T] and W^T [in x out]
            return operand_bytes(in_features, T) + operand_bytes(in_features, out_features);
        case MXFP4_LAYER_FORWARD:    // X [T x in] and W [out x in]
            return operand_bytes(T, in_features) + operand_bytes(out_features, in_features);
        case MXFP4_LAYER_BACKWARD:   // dY [T x out] and dY^T [out x T]
            return operand_bytes(T, out_features) + operand_bytes(out_features, T);
        default: return 0;
    }
}

static int layer_args_ok(int64_t T, int64_t in_f, int64_t out_f, int hmode, int rounding, const void* saved,
                         size_t saved_bytes, const void* workspace, size_t workspace_bytes, int ws_kind)
{
    if (T <= 0 || in_f <= 0 || out_f <= 0) return MXFP4_ERR_SHAPE;
    if (T % 32 != 0 || in_f % 32 != 0 || out_f % 32 != 0) return MXFP4_ERR_SHAPE;
    if (T > 0x7FFFFFFF || in_f > 0x7FFFFFFF || out_f > 0x7FFFFFFF) return MXFP4_ERR_SHAPE;
    if (!quant_tiles_fit(T, in_f) || !quant_tiles_fit(out_f, in_f) || !quant_tiles_fit(T, out_f) ||
        !gemm_tiles_fit(T, out_f, in_f) || !gemm_tiles_fit(T, in_f, out_f) || !gemm_tiles_fit(out_f, in_f, T))
        return MXFP4_ERR_SHAPE;
    if (hmode < 0 || hmode > 4 || rounding < 0 || rounding > 1) return MXFP4_ERR_ENUM;
    if (!saved || saved_bytes < mxfp4_linear_layer_bytes(T, in_f, out_f, MXFP4_LAYER_SAVED)) return MXFP4_ERR_WORKSPACE;
    if (!workspace || workspace_bytes < mxfp4_linear_layer_bytes(T, in_f, out_f, ws_kind)) return MXFP4_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(saved) & 255u) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return MXFP4_ERR_ALIGN;
    return MXFP4_OK;
}

static float rotation_alpha(int hmode)
{
    // H * H^T = n * I for the +-1 matrix of order n: undone exactly in the GEMM epilogue
    return hmode == MXFP4_HADAMARD_NONE ? 1.0f : (hmode <= MXFP4_HADAMARD_RAND ? 0.03125f : 0.0625f);
}

// Optional stream ordering around the three launches of a forward or backward call, used by the
// host-buffer form to tie each launch to the copy that feeds it or drains it: `wait[i]` (if set)
// is waited for on the stream before launch i, `done[i]` (if set) is recorded after it.
struct LaunchHooks {
    cudaEvent_t wait[3];
    cudaEvent_t done[3];
};

static int hook_wait(const LaunchHooks* h, int i, cudaStream_t st)
{
    if (h && h->wait[i] && cudaStreamWaitEvent(st, h->wait[i], 0) != cudaSuccess) return MXFP4_ERR_CUDA;
    return MXFP4_OK;
}

static int hook_done(const LaunchHooks* h, int i, cudaStream_t st)
{
    if (h && h->done[i] && cudaEventRecord(h->done[i], st) != cudaSuccess) return MXFP4_ERR_CUDA;
    return MXFP4_OK;
}

// mxfp4_linear_forward; launches: 0 = quantize X, 1 = quantize W, 2 = Fprop GEMM.
static int linear_forward_impl(const void* X, const void* W, void* Y, int64_t T, int64_t in_features,
                               int64_t out_features, int hadamard_mode, int rounding, uint64_t seed, int out_dtype,
                               void* saved, size_t saved_bytes, void* workspace, size_t workspace_bytes, void* stream,
                               const LaunchHooks* hooks)
{
    if (!X || !W || !Y) return MXFP4_ERR_NULL;
    if (out_dtype != MXFP4_OUT_BF16 && out_dtype != MXFP4_OUT_FP32) return MXFP4_ERR_ENUM;
    if (!aligned16(X) || !aligned16(W) || !aligned16(Y)) return MXFP4_ERR_ALIGN;
    int rc = layer_args_ok(T, in_features, out_features, hadamard_mode, rounding, saved, saved_bytes, workspace,
                           workspace_bytes, MXFP4_LAYER_FORWARD);
    if (rc != MXFP4_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    uint8_t* x_codes = ws;
    uint8_t* x_scales = x_codes + round_up(mxfp4_codes_bytes(T, in_features), 256);
    uint8_t* w_codes = ws + operand_bytes(T, in_features);
    uint8_t* w_scales = w_codes + round_up(mxfp4_codes_bytes(out_features, in_features), 256);
    uint8_t* sv = static_cast<uint8_t*>(saved);
    uint8_t* xt_codes = sv;
    uint8_t* xt_scales = xt_codes + round_up(mxfp4_codes_bytes(in_features, T), 256);
    uint8_t* wt_codes = sv + operand_bytes(in_features, T);
    uint8_t* wt_scales = wt_codes + round_up(mxfp4_codes_bytes(in_features, out_features), 256);
    // tags as in the per-pass entry points: A operands 0, B operands 1 (X^T is Wgrad's B, W^T Dgrad's B)
    if ((rc = hook_wait(hooks, 0, st)) != MXFP4_OK) return rc;
    rc = mxfp4_quantize_dual(X, T, in_features, in_features, hadamard_mode, rounding, seed, 0u, 1u,
                             MXFP4_BLOCK_1X32, x_codes, x_scales, xt_codes, xt_scales, MXFP4_SCALES_TILED, stream);
    if (rc != MXFP4_OK) return rc;
    if ((rc = hook_done(hooks, 0, st)) != MXFP4_OK || (rc = hook_wait(hooks, 1, st)) != MXFP4_OK) return rc;
    rc = mxfp4_quantize_dual(W, out_features, in_features, in_features, hadamard_mode, rounding, seed, 1u, 1u,
                             MXFP4_BLOCK_1X32, w_codes, w_scales, wt_codes, wt_scales, MXFP4_SCALES_TILED, stream);
    if (rc != MXFP4_OK) return rc;
    if ((rc = hook_done(hooks, 1, st)) != MXFP4_OK || (rc = hook_wait(hooks, 2, st)) != MXFP4_OK) return rc;
    rc = mxfp4_gemm(x_codes, x_scales, w_codes, w_scales, T, out_features, in_features,
                    rotation_alpha(hadamard_mode), Y, out_dtype, out_features, nullptr, 0, stream);
    if (rc != MXFP4_OK) return rc;
    return hook_done(hooks, 2, st);
}

int mxfp4_linear_forward(const void* X, const void* W, void* Y, int64_t T, int64_t in_features,
                         int64_t out_features, int hadamard_mode, int rounding, uint64_t seed, int out_dtype,
                         void* saved, size_t saved_bytes, void* workspace, size_t workspace_bytes, void* stream)
{
    return linear_forward_impl(X, W, Y, T, in_features, out_features, hadamard_mode, rounding, seed, out_dtype, saved,
                               saved_bytes, workspace, workspace_bytes, stream, nullptr);
}

// mxfp4_linear_backward; launches: 0 = quantize dY, 1 = Dgrad GEMM, 2 = Wgrad GEMM.
static int linear_backward_impl(const void* dY, void* dX, void* dW, int64_t T, int64_t in_features,
                                int64_t out_features, int hadamard_mode, int rounding, uint64_t seed, int dx_dtype,
                                int dw_dtype, const void* saved, size_t saved_bytes, void* workspace,
                                size_t workspace_bytes, void* stream, const LaunchHooks* hooks)
{
    if (!dY || !dX || !dW) return MXFP4_ERR_NULL;
    for (int d : {dx_dtype, dw_dtype})
        if (d != MXFP4_OUT_BF16 && d != MXFP4_OUT_FP32) return MXFP4_ERR_ENUM;
    if (!aligned16(dY) || !aligned16(dX) || !aligned16(dW)) return MXFP4_ERR_ALIGN;
    int rc = layer_args_ok(T, in_features, out_features, hadamard_mode, rounding, saved, saved_bytes, workspace,
                           workspace_bytes, MXFP4_LAYER_BACKWARD);
    if (rc != MXFP4_OK) return rc;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    uint8_t* dy_codes = ws;
    uint8_t* dy_scales = dy_codes + round_up(mxfp4_codes_bytes(T, out_features), 256);
    uint8_t* dyt_codes = ws + operand_bytes(T, out_features);
    uint8_t* dyt_scales = dyt_codes + round_up(mxfp4_codes_bytes(out_features, T), 256);
    const uint8_t* sv = static_cast<const uint8_t*>(saved);
    const uint8_t* xt_codes = sv;
    const uint8_t* xt_scales = xt_codes + round_up(mxfp4_codes_bytes(in_features, T), 256);
    const uint8_t* wt_codes = sv + operand_bytes(in_features, T);
    const uint8_t* wt_scales = wt_codes + round_up(mxfp4_codes_bytes(in_features, out_features), 256);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((rc = hook_wait(hooks, 0, st)) != MXFP4_OK) return rc;
    rc = mxfp4_quantize_dual(dY, T, out_features, out_features, hadamard_mode, rounding, seed, 0u, 0u,
                             MXFP4_BLOCK_1X32, dy_codes, dy_scales, dyt_codes, dyt_scales, MXFP4_SCALES_TILED, stream);
    if (rc != MXFP4_OK) return rc;
    if ((rc = hook_done(hooks, 0, st)) != MXFP4_OK || (rc = hook_wait(hooks, 1, st)) != MXFP4_OK) return rc;
    const float alpha = rotation_alpha(hadamard_mode);
    // dX [T x in] = dY [T x out] . (W^T operand [in x out])^T
    rc = mxfp4_gemm(dy_codes, dy_scales, wt_codes, wt_scales, T, in_features, out_features, alpha, dX, dx_dtype,
                    in_features, nullptr, 0, stream);
    if (rc != MXFP4_OK) return rc;
    if ((rc = hook_done(hooks, 1, st)) != MXFP4_OK || (rc = hook_wait(hooks, 2, st)) != MXFP4_OK) return rc;
    // dW [out x in] = dY^T [out x T] . (X^T operand [in x T])^T
    rc = mxfp4_gemm(dyt_codes, dyt_scales, xt_codes, xt_scales, out_features, in_features, T, alpha, dW, dw_dtype,
                    in_features, nullptr, 0, stream);
    if (rc != MXFP4_OK) return rc;
    return hook_done(hooks, 2, st);
}

int mxfp4_linear_backward(const void* dY, void* dX, void* dW, int64_t T, int64_t in_features,
                          int64_t out_features, int hadamard_mode, int rounding, uint64_t seed, int dx_dtype,
                          int dw_dtype, const void* saved, size_t saved_bytes, void* workspace,
                          size_t workspace_bytes, void* stream)
{
    return linear_backward_impl(dY, dX, dW, T, in_features, out_features, hadamard_mode, rounding, seed, dx_dtype,
                                dw_dtype, saved, saved_bytes, workspace, workspace_bytes, stream, nullptr);
}

// Copy streams and events of the host-buffer layer call, one set per device, created on first
// use and kept for the life of the process.
struct HostPipe {
    cudaStream_t h2d, d2h;
    // per tensor t in (X, W, dY): in[t] = its copy to the device has landed, read[t] = the quantize
    // launch that reads its staging buffer is done (the buffer may be overwritten);
    // per result r in (Y, dX, dW): ready[r] = its GEMM is done, out[r] = its copy to the host is
    // done (the staging buffer may be overwritten)
    cudaEvent_t in[3], read[3], ready[3], out[3];
    bool ok;
};

static int host_pipe(HostPipe** out)
{
    static HostPipe pipes[kMaxDevices] = {};
    static PerDeviceOnce once;
    const int dev = current_device();
    if (dev < 0) return MXFP4_ERR_CUDA;
    HostPipe& p = pipes[dev];
    *out = &p;
    return once.run(dev, [&] {
        if (cudaStreamCreateWithFlags(&p.h2d, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&p.d2h, cudaStreamNonBlocking) != cudaSuccess)
            return MXFP4_ERR_CUDA;
        for (cudaEvent_t* set : {p.in, p.read, p.ready, p.out})
            for (int i = 0; i < 3; ++i)
                if (cudaEventCreateWithFlags(&set[i], cudaEventDisableTiming) != cudaSuccess) return MXFP4_ERR_CUDA;
        p.ok = true;
        return MXFP4_OK;
    });
}

int mxfp4_linear_layer_host_drain(void* stream);

int mxfp4_linear_layer_host(const void* X_host, const void* W_host, const void* dY_host, void* Y_host,
                            void* dX_host, void* dW_host, int64_t T, int64_t in_features, int64_t out_features,
                            int hadamard_mode, int rounding, uint64_t seed, int y_dtype, int dx_dtype, int dw_dtype,
                            void* dev_x, void* dev_w, void* dev_dy, void* dev_y, void* dev_dx, void* dev_dw,
                            void* saved, size_t saved_bytes, void* workspace, size_t workspace_bytes, void* stream,
                            int drain)
{
    if (!X_host || !W_host || !dY_host || !Y_host || !dX_host || !dW_host) return MXFP4_ERR_NULL;
    if (!dev_x || !dev_w || !dev_dy || !dev_y || !dev_dx || !dev_dw) return MXFP4_ERR_NULL;
    for (int d : {y_dtype, dx_dtype, dw_dtype})
        if (d != MXFP4_OUT_BF16 && d != MXFP4_OUT_FP32) return MXFP4_ERR_ENUM;
    int rc = layer_args_ok(T, in_features, out_features, hadamard_mode, rounding, saved, saved_bytes, workspace,
                           workspace_bytes, MXFP4_LAYER_FORWARD);
    if (rc != MXFP4_OK) return rc;
    if (workspace_bytes < mxfp4_linear_layer_bytes(T, in_features, out_features, MXFP4_LAYER_BACKWARD))
        return MXFP4_ERR_WORKSPACE;
    for (const void* q : {static_cast<const void*>(dev_x), static_cast<const void*>(dev_w),
                          static_cast<const void*>(dev_dy), static_cast<const void*>(dev_y),
                          static_cast<const void*>(dev_dx), static_cast<const void*>(dev_dw)})
        if (!aligned16(q)) return MXFP4_ERR_ALIGN;      // before the first copy is enqueued
    HostPipe* hp = nullptr;
    rc = host_pipe(&hp);
    if (rc != MXFP4_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t x_bytes = static_cast<size_t>(T) * in_features * 2;
    const size_t w_bytes = static_cast<size_t>(out_features) * in_features * 2;
    const size_t dy_bytes = static_cast<size_t>(T) * out_features * 2;
    const size_t y_out = static_cast<size_t>(T) * out_features * (y_dtype == MXFP4_OUT_BF16 ? 2 : 4);
    const size_t dx_out = static_cast<size_t>(T) * in_features * (dx_dtype == MXFP4_OUT_BF16 ? 2 : 4);
    const size_t dw_out = static_cast<size_t>(out_features) * in_features * (dw_dtype == MXFP4_OUT_BF16 ? 2 : 4);
#define MXFP4_TRY(call) do { if ((call) != cudaSuccess) return MXFP4_ERR_CUDA; } while (0)
    // Inputs travel on their own stream in the order they are needed.  A staging buffer is
    // overwritten as soon as the quantize launch of the PREVIOUS call that read it is done -- not
    // when that whole call is -- so the next layer's inputs flow in while this layer's GEMMs run
    // (waiting on an event that was never recorded is a no-op: the first call).
    const void* src[3] = {X_host, W_host, dY_host};
    void* stg_in[3] = {dev_x, dev_w, dev_dy};
    const size_t in_bytes[3] = {x_bytes, w_bytes, dy_bytes};
    for (int i = 0; i < 3; ++i) {
        MXFP4_TRY(cudaStreamWaitEvent(hp->h2d, hp->read[i], 0));
        MXFP4_TRY(cudaMemcpyAsync(stg_in[i], src[i], in_bytes[i], cudaMemcpyHostToDevice, hp->h2d));
        MXFP4_TRY(cudaEventRecord(hp->in[i], hp->h2d));
    }
    // Compute on the caller's stream: each quantize launch waits for its tensor, each GEMM for the
    // previous call's copy out of the staging buffer it is about to overwrite.
    const LaunchHooks fwd = {{hp->in[0], hp->in[1], hp->out[0]}, {hp->read[0], hp->read[1], hp->ready[0]}};
    rc = linear_forward_impl(dev_x, dev_w, dev_y, T, in_features, out_features, hadamard_mode, rounding, seed, y_dtype,
                             saved, saved_bytes, workspace, workspace_bytes, stream, &fwd);
    if (rc != MXFP4_OK) return rc;
    const LaunchHooks bwd = {{hp->in[2], hp->out[1], hp->out[2]}, {hp->read[2], hp->ready[1], hp->ready[2]}};
    rc = linear_backward_impl(dev_dy, dev_dx, dev_dw, T, in_features, out_features, hadamard_mode, rounding, seed,
                              dx_dtype, dw_dtype, saved, saved_bytes, workspace, workspace_bytes, stream, &bwd);
    if (rc != MXFP4_OK) return rc;
    // results leave on a third stream, each as soon as its GEMM is done, while later inputs still arrive
    void* dst[3] = {Y_host, dX_host, dW_host};
    const void* stg_out[3] = {dev_y, dev_dx, dev_dw};
    const size_t out_bytes[3] = {y_out, dx_out, dw_out};
    for (int i = 0; i < 3; ++i) {
        MXFP4_TRY(cudaStreamWaitEvent(hp->d2h, hp->ready[i], 0));
        MXFP4_TRY(cudaMemcpyAsync(dst[i], stg_out[i], out_bytes[i], cudaMemcpyDeviceToHost, hp->d2h));
        MXFP4_TRY(cudaEventRecord(hp->out[i], hp->d2h));
    }
#undef MXFP4_TRY
    return drain ? mxfp4_linear_layer_host_drain(stream) : MXFP4_OK;
}

int mxfp4_linear_layer_host_drain(void* stream)
{
    HostPipe* hp = nullptr;
    const int rc = host_pipe(&hp);
    if (rc != MXFP4_OK) return rc;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess ||
        cudaStreamSynchronize(hp->h2d) != cudaSuccess || cudaStreamSynchronize(hp->d2h) != cudaSuccess)
        return MXFP4_ERR_CUDA;
    return MXFP4_OK;
}

int mxfp4_linear_host(int pass, const void* a_host, const void* b_host, void* out_host, int64_t T,
                      int64_t in_features, int64_t out_features, int hadamard_mode, int rounding,
                      uint64_t seed, int out_dtype, void* dev_a, void* dev_b, void* dev_out,
                      void* workspace, size_t workspace_bytes, void* stream)
{
    if (pass < 0 || pass > 2) return MXFP4_ERR_ENUM;
    if (!a_host || !b_host || !out_host || !dev_a || !dev_b || !dev_out) return MXFP4_ERR_NULL;
    if (out_dtype != MXFP4_OUT_BF16 && out_dtype != MXFP4_OUT_FP32) return MXFP4_ERR_ENUM;
    if (T <= 0 || in_features <= 0 || out_features <= 0) return MXFP4_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // source shapes: (a, b, out) = (X, W, Y) / (dY, W, dX) / (dY, X, dW)
    const size_t a_elems = static_cast<size_t>(T) * (pass == MXFP4_PASS_FPROP ? in_features : out_features);
    const size_t b_elems = pass == MXFP4_PASS_WGRAD ? static_cast<size_t>(T) * in_features
                                                    : static_cast<size_t>(out_features) * in_features;
    int64_t M, N, K;
    linear_dims(pass, T, in_features, out_features, &M, &N, &K);
    const size_t out_bytes = static_cast<size_t>(M) * N * (out_dtype == MXFP4_OUT_BF16 ? 2 : 4);
    // argument errors are reported before the first copy is enqueued
    const int vrc = linear_pass(pass, dev_a, dev_b, dev_out, T, in_features, out_features, hadamard_mode, rounding,
                                seed, out_dtype, workspace, workspace_bytes, stream, MXFP4_PRECISION_MXFP4, true);
    if (vrc != MXFP4_OK) return vrc;
    if (cudaMemcpyAsync(dev_a, a_host, a_elems * 2, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(dev_b, b_host, b_elems * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return MXFP4_ERR_CUDA;
    const int rc = linear_pass(pass, dev_a, dev_b, dev_out, T, in_features, out_features,
                               hadamard_mode, rounding, seed, out_dtype, workspace, workspace_bytes,
                               stream);
    if (rc != MXFP4_OK) return rc;
    if (cudaMemcpyAsync(out_host, dev_out, out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return MXFP4_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? MXFP4_OK : MXFP4_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------
// Allocation-free variant of the fused passes.  The scratch the passes need (the two quantized
// operands) lives in this file-scope device array instead of a caller-supplied workspace.  In
// host code the array's name is only a stand-in for the symbol, not a device address, so the
// address is fetched once per device with cudaGetSymbolAddress and cached.
static __device__ __align__(256) uint8_t g_static_scratch[MXFP4_STATIC_SCRATCH_BYTES];

static int static_scratch_address(uint8_t** out)
{
    static uint8_t* cached[kMaxDevices] = {};
    static PerDeviceOnce once;
    const int dev = current_device();
    if (dev < 0) return MXFP4_ERR_CUDA;
    const int rc = once.run(dev, [&] {
        uint8_t* ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_scratch) != cudaSuccess || !ptr)
            return MXFP4_ERR_CUDA;
        cached[dev] = ptr;
        return MXFP4_OK;
    });
    *out = cached[dev];
    return rc;
}

int mxfp4_linear_static(int pass, const void* a, const void* b, void* out, int64_t T,
                        int64_t in_features, int64_t out_features, int hadamard_mode, int rounding,
                        uint64_t seed, int out_dtype, void* stream)
{
    if (pass < 0 || pass > 2) return MXFP4_ERR_ENUM;
    if (T <= 0 || in_features <= 0 || out_features <= 0) return MXFP4_ERR_SHAPE;
    int64_t M, N, K;
    linear_dims(pass, T, in_features, out_features, &M, &N, &K);
    if (K % 32 != 0) return MXFP4_ERR_SHAPE;
    const size_t need = mxfp4_linear_workspace_bytes(T, in_features, out_features, pass);
    if (need == 0) return MXFP4_ERR_SHAPE;
    if (need > static_cast<size_t>(MXFP4_STATIC_SCRATCH_BYTES)) return MXFP4_ERR_STATIC_LIMIT;
    uint8_t* scratch = nullptr;
    const int rc = static_scratch_address(&scratch);
    if (rc != MXFP4_OK) return rc;
    // Nothing in the scratch has to start at zero: the two quantize launches of this call
    // rewrite every code byte and every scale tile (padding included) the GEMM will read.
    return linear_pass(pass, a, b, out, T, in_features, out_features, hadamard_mode, rounding, seed,
                       out_dtype, scratch, MXFP4_STATIC_SCRATCH_BYTES, stream);
}

int mxfp4_selftest_wait_timeout(void* stream)
{
    const DeviceInfo& dev = device_info();
    if (!dev.ok) return MXFP4_ERR_CUDA;
    if (dev.cc_major != 10) return MXFP4_ERR_DEVICE;
    selftest_wait_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>();
    return cudaGetLastError() == cudaSuccess ? MXFP4_OK : MXFP4_ERR_CUDA;
}

int mxfp4_probe_mma_rate(int iterations, int random_operands, void* stream, double* flops)
{
    if (iterations <= 0 || iterations > 20000) return MXFP4_ERR_SHAPE;   // a launch stays within ~10 ms
    const DeviceInfo& dev = device_info();
    if (!dev.ok) return MXFP4_ERR_CUDA;
    if (dev.cc_major != 10) return MXFP4_ERR_DEVICE;
    const size_t smem = sizeof(MmaProbeSmem) + 1024;
    static PerDeviceOnce once;
    const int rc = ensure_smem_attribute(once, mma_rate_probe_kernel, smem);
    if (rc != MXFP4_OK) return rc;
    const int clusters = dev.sm_count / 2;
    mma_rate_probe_kernel<<<2 * clusters, kMmaProbeThreads, smem, static_cast<cudaStream_t>(stream)>>>(
        iterations, random_operands ? 1 : 0);
    if (cudaGetLastError() != cudaSuccess) return MXFP4_ERR_CUDA;
    if (flops) *flops = 2.0 * kPTileM * kPMmaN * 64.0 * 8.0 * iterations * clusters;
    return MXFP4_OK;
}

int mxfp4_bounds_checked(void)
{
#ifdef MXFP4_BOUNDS
    return 1;
#else
    return 0;
#endif
}

int mxfp4_selftest_bounds(void* stream)
{
    const DeviceInfo& dev = device_info();
    if (!dev.ok) return MXFP4_ERR_CUDA;
    if (dev.cc_major != 10) return MXFP4_ERR_DEVICE;
    selftest_bounds_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>();
    return cudaGetLastError() == cudaSuccess ? MXFP4_OK : MXFP4_ERR_CUDA;
}

int mxfp4_check(void* stream)
{
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return MXFP4_ERR_CUDA;
    int status = 0;
    if (cudaMemcpyFromSymbol(&status, g_device_status, sizeof(int)) != cudaSuccess)
        return MXFP4_ERR_CUDA;
    if (status != 0) {
        const int zero = 0;
        cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int));
    }
    return status;
}

}  // extern "C"
