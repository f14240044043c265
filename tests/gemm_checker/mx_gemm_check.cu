// Slow fp64 checker for the block-scaled MXFP4 GEMM's FULL output (test infrastructure).
//
// What it computes is the plain definition (Appendix A.1 Eq. (1) operands, Appendix C products):
//   ref[m][n] = alpha * sum_t 2^(sa[m][t] - 127) * 2^(sb[n][t] - 127) * sum_{k in block t} val(a[m][k]) * val(b[n][k])
//   S[m][n]   = |alpha| * sum of the absolute values of the same products
// with val(code) the E2M1 value of a 4-bit code, one thread per output element, no tensor cores,
// integer products (exact: every E2M1 value is a multiple of 1/2) and fp64 accumulation over the
// blocks.  It shares nothing with the library under test: no header, no kernel, no table.  It is
// itself checked against the CPU oracle on sampled rows before its verdict on a whole output is
// trusted.  Operands: codes [rows x K/2] bytes (element k even in the low nibble), scales in the
// canonical layout [rows x K/32] bytes, all device pointers.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

constexpr int kTile = 16;        // outputs per block edge
constexpr int kChunkBlocks = 8;  // MX blocks of K per shared-memory chunk (256 elements = 128 bytes per row)

// twice the E2M1 value of a code's magnitude bits
__device__ __forceinline__ int twice_value(int code)
{
    const int mag = code & 7;
    const int v = mag < 4 ? mag : (mag == 4 ? 4 : (mag == 5 ? 6 : (mag == 6 ? 8 : 12)));
    return (code & 8) ? -v : v;
}

struct Verdict {
    unsigned long long n_bad;      // elements out of tolerance (or not finite)
    unsigned long long first_bad;  // m * N + n of the smallest offending index seen (not exact under races; diagnostic)
    double worst;                  // largest |out - ref| / tolerance
};

__device__ double atomic_max_double(double* addr, double v)
{
    unsigned long long* p = reinterpret_cast<unsigned long long*>(addr);
    unsigned long long old = *p, assumed;
    do {
        assumed = old;
        if (__longlong_as_double(static_cast<long long>(assumed)) >= v) break;
        old = atomicCAS(p, assumed, static_cast<unsigned long long>(__double_as_longlong(v)));
    } while (assumed != old);
    return v;
}

__global__ void check_kernel(const uint8_t* __restrict__ a_codes, const uint8_t* __restrict__ a_scales,
                             const uint8_t* __restrict__ b_codes, const uint8_t* __restrict__ b_scales, long long M,
                             long long N, long long K, double alpha, const void* out, int out_is_bf16, long long ld_out,
                             double rel_tol, double bf16_term, double* ref_out, double* s_out, Verdict* verdict)
{
    // decoded operands of the chunk: twice the E2M1 value of every element, as signed bytes
    // (rows padded by four bytes so that the sixteen rows a warp reads fall into different banks)
    __shared__ __align__(16) int8_t sa_val[kTile][kChunkBlocks * 32 + 4];
    __shared__ __align__(16) int8_t sb_val[kTile][kChunkBlocks * 32 + 4];
    __shared__ uint8_t sa_scale[kTile][kChunkBlocks];
    __shared__ uint8_t sb_scale[kTile][kChunkBlocks];
    const int tx = threadIdx.x, ty = threadIdx.y;
    const long long m = static_cast<long long>(blockIdx.y) * kTile + ty;
    const long long n = static_cast<long long>(blockIdx.x) * kTile + tx;
    const long long nt = K / 32;
    double acc = 0.0, sabs = 0.0;
    for (long long t0 = 0; t0 < nt; t0 += kChunkBlocks) {
        const int nb = static_cast<int>(nt - t0 < kChunkBlocks ? nt - t0 : kChunkBlocks);
        // cooperative load and decode: 16 rows x up to 128 code bytes per operand
        const int tid = ty * kTile + tx;
        for (int i = tid; i < kTile * kChunkBlocks * 16; i += kTile * kTile) {
            const int r = i / (kChunkBlocks * 16), c = i % (kChunkBlocks * 16);
            const long long ra = static_cast<long long>(blockIdx.y) * kTile + r;
            const long long rb = static_cast<long long>(blockIdx.x) * kTile + r;
            const bool in_k = c < nb * 16;
            const int ca = (ra < M && in_k) ? a_codes[ra * (K / 2) + t0 * 16 + c] : 0;
            const int cb = (rb < N && in_k) ? b_codes[rb * (K / 2) + t0 * 16 + c] : 0;
            sa_val[r][2 * c] = static_cast<int8_t>(twice_value(ca & 15));       // element k even: low nibble
            sa_val[r][2 * c + 1] = static_cast<int8_t>(twice_value(ca >> 4));
            sb_val[r][2 * c] = static_cast<int8_t>(twice_value(cb & 15));
            sb_val[r][2 * c + 1] = static_cast<int8_t>(twice_value(cb >> 4));
        }
        for (int i = tid; i < kTile * kChunkBlocks; i += kTile * kTile) {
            const int r = i / kChunkBlocks, c = i % kChunkBlocks;
            const long long ra = static_cast<long long>(blockIdx.y) * kTile + r;
            const long long rb = static_cast<long long>(blockIdx.x) * kTile + r;
            sa_scale[r][c] = (ra < M && c < nb) ? a_scales[ra * nt + t0 + c] : 0;
            sb_scale[r][c] = (rb < N && c < nb) ? b_scales[rb * nt + t0 + c] : 0;
        }
        __syncthreads();
        for (int b = 0; b < nb; ++b) {
            int dot = 0, dabs = 0;               // in units of 1/4; |dot| <= 32 * 144
            for (int j = 0; j < 32; j += 4) {    // four elements per step: integer dot products of signed bytes
                const int va = *reinterpret_cast<const int*>(&sa_val[ty][b * 32 + j]);
                const int vb = *reinterpret_cast<const int*>(&sb_val[tx][b * 32 + j]);
                dot = __dp4a(va, vb, dot);
                dabs = __dp4a(static_cast<int>(__vabsss4(va)), static_cast<int>(__vabsss4(vb)), dabs);
            }
            // 2^(sa - 127) * 2^(sb - 127) / 4, exact in fp64 for every pair of E8M0 bytes
            const double scale = ldexp(1.0, static_cast<int>(sa_scale[ty][b]) + static_cast<int>(sb_scale[tx][b]) - 256);
            acc += scale * static_cast<double>(dot);
            sabs += scale * static_cast<double>(dabs);
        }
        __syncthreads();
    }
    if (m >= M || n >= N) return;
    const double ref = alpha * acc;
    const double S = fabs(alpha) * sabs;
    if (ref_out) {
        ref_out[m * N + n] = ref;
        s_out[m * N + n] = S;
    }
    if (out) {
        double got;
        if (out_is_bf16)
            got = static_cast<double>(__bfloat162float(static_cast<const __nv_bfloat16*>(out)[m * ld_out + n]));
        else
            got = static_cast<double>(static_cast<const float*>(out)[m * ld_out + n]);
        const double tol = rel_tol * S + bf16_term * fabs(ref) + 1e-38;
        const double err = fabs(got - ref);
        const bool bad = !(err <= tol);          // a NaN fails
        if (bad) {
            atomicAdd(&verdict->n_bad, 1ull);
            atomicMin(&verdict->first_bad, static_cast<unsigned long long>(m * N + n));
        }
        if (err == err) atomic_max_double(&verdict->worst, err / tol);
    }
}

}  // namespace

// Compares out[M x N] (bf16 or fp32, leading dimension ld_out) with the fp64 definition, element
// by element: |out - ref| <= rel_tol * S + bf16_term * |ref|.  verdict_host receives
// {n_bad, first_bad_index, worst_ratio_bits}.  ref_out / s_out (optional, device, [M x N] doubles)
// receive the reference and S; out may be NULL when only those are wanted.  Synchronous.
// Returns 0, or a negative number for a bad argument / CUDA error.
extern "C" int mxcheck_gemm(const void* a_codes, const void* a_scales, const void* b_codes, const void* b_scales,
                            long long M, long long N, long long K, double alpha, const void* out, int out_is_bf16,
                            long long ld_out, double rel_tol, double bf16_term, double* ref_out, double* s_out,
                            unsigned long long* verdict_host)
{
    if (!a_codes || !a_scales || !b_codes || !b_scales || !verdict_host) return -1;
    if (M <= 0 || N <= 0 || K <= 0 || K % 32 != 0) return -2;
    Verdict* dv = nullptr;
    if (cudaMalloc(&dv, sizeof(Verdict)) != cudaSuccess) return -3;
    Verdict init = {0ull, ~0ull, 0.0};
    cudaMemcpy(dv, &init, sizeof(init), cudaMemcpyHostToDevice);
    dim3 grid(static_cast<unsigned>((N + kTile - 1) / kTile), static_cast<unsigned>((M + kTile - 1) / kTile));
    check_kernel<<<grid, dim3(kTile, kTile)>>>(static_cast<const uint8_t*>(a_codes), static_cast<const uint8_t*>(a_scales),
                                               static_cast<const uint8_t*>(b_codes), static_cast<const uint8_t*>(b_scales),
                                               M, N, K, alpha, out, out_is_bf16, ld_out, rel_tol, bf16_term, ref_out, s_out, dv);
    int rc = 0;
    if (cudaGetLastError() != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) rc = -4;
    Verdict v = init;
    if (rc == 0 && cudaMemcpy(&v, dv, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess) rc = -4;
    cudaFree(dv);
    verdict_host[0] = v.n_bad;
    verdict_host[1] = v.first_bad;
    static_assert(sizeof(double) == sizeof(unsigned long long), "");
    __builtin_memcpy(&verdict_host[2], &v.worst, sizeof(double));
    return rc;
}
