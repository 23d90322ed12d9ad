// The native FP64 path for out-of-range rows (Algorithm 1, last line: "native-FP64 fallback for
// out-of-range rows"; Algorithm 3: "ESC range check; re-issue out-of-range rows on the native-FP64
// path").  The paper names the step and leaves its arithmetic open; the reading taken here:
// every entry of a re-issued row is the compensated inner product of its row of A and column of B,
//     for kk = 0 .. k-1:   p = a b,  pe = fma(a, b, -p)            (a b = p + pe exactly)
//                          s = acc + p,  se = its exact rounding error (error-free sum)
//                          comp += pe + se,  acc = s
//     P = acc + comp,
// FP64 operations only, in this order, so that the value is a function of the data alone (no
// dependence on tiling or on the number of threads) and meets the same 2u (|A||B|) contract as the
// emulated rows.  C(i,j) = alpha P (beta = 0) or C(i,j) + alpha P (beta = 1) from the caller's old
// C: the reconstruction leaves the re-issued rows untouched.
//
// Work distribution: the re-issued rows come as an ascending list; a thread block takes 64 of
// them x 64 columns, stages 16 inner indices at a time in shared memory, and each thread carries a
// 4 x 4 block of (acc, comp) pairs.  The grid is sized for the worst case (every row re-issued),
// blocks beyond the list's end return at once: the number of rows is known on the device only.
#include "oz_internal.h"

namespace oz {
namespace {

constexpr int kFbRows = 64, kFbCols = 64, kFbK = 16, kFbThreads = 256;

__global__ void __launch_bounds__(kFbThreads)
native_rows_kernel(int64_t m, int64_t n, int64_t k, const double *__restrict__ A, int64_t lda,
                   const double *__restrict__ B, int64_t ldb, const int *__restrict__ list,
                   const unsigned int *__restrict__ count, const int32_t *__restrict__ shiftB,
                   double alpha, double beta, double *__restrict__ C, int64_t ldc)
{
    const int64_t rows = *count;
    const int64_t r0 = static_cast<int64_t>(blockIdx.y) * kFbRows;
    if (r0 >= rows) return;
    const int64_t c0 = static_cast<int64_t>(blockIdx.x) * kFbCols;
    __shared__ __align__(16) double As[kFbK][kFbRows + 2];     // +2: rows stay 16-byte aligned for the pair loads
    __shared__ __align__(16) double Bs[kFbK][kFbCols + 2];
    __shared__ int64_t row_of[kFbRows];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    if (tid < kFbRows) row_of[tid] = r0 + tid < rows ? list[r0 + tid] : -1;
    __syncthreads();

    double acc[4][4], comp[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = comp[r][c] = 0.0;

    for (int64_t k0 = 0; k0 < k; k0 += kFbK) {
        const int kn = k - k0 < kFbK ? static_cast<int>(k - k0) : kFbK;
        // A: consecutive threads take consecutive re-issued rows of one inner index
#pragma unroll
        for (int u = 0; u < kFbRows * kFbK / kFbThreads; ++u) {
            const int r = tid & (kFbRows - 1), kk = (tid >> 6) + 4 * u;
            const int64_t row = row_of[r];
            As[kk][r] = (row >= 0 && kk < kn) ? A[row + (k0 + kk) * lda] : 0.0;
        }
        // B: consecutive threads take consecutive inner indices of one column
#pragma unroll
        for (int u = 0; u < kFbCols * kFbK / kFbThreads; ++u) {
            const int kk = tid & (kFbK - 1), c = (tid >> 4) + 16 * u;
            Bs[kk][c] = (c0 + c < n && kk < kn) ? B[(k0 + kk) + (c0 + c) * ldb] : 0.0;
        }
        __syncthreads();
        for (int kk = 0; kk < kn; ++kk) {
            const double2 a01 = *reinterpret_cast<const double2 *>(&As[kk][ty * 4]);
            const double2 a23 = *reinterpret_cast<const double2 *>(&As[kk][ty * 4 + 2]);
            const double2 b01 = *reinterpret_cast<const double2 *>(&Bs[kk][tx * 4]);
            const double2 b23 = *reinterpret_cast<const double2 *>(&Bs[kk][tx * 4 + 2]);
            const double a[4] = {a01.x, a01.y, a23.x, a23.y}, b[4] = {b01.x, b01.y, b23.x, b23.y};
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const double p = __dmul_rn(a[r], b[c]);
                    const double pe = __fma_rn(a[r], b[c], -p);
                    const double s = __dadd_rn(acc[r][c], p);
                    const double bb = __dsub_rn(s, acc[r][c]);
                    const double se = __dadd_rn(__dsub_rn(acc[r][c], __dsub_rn(s, bb)), __dsub_rn(p, bb));
                    comp[r][c] = __dadd_rn(comp[r][c], __dadd_rn(pe, se));
                    acc[r][c] = s;
                }
        }
        __syncthreads();
    }

    const double nan = __longlong_as_double(0x7FF8000000000000ll);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int64_t j = c0 + tx * 4 + c;
        if (j >= n) continue;
        const bool bad = shiftB[j] == OZ_NONFINITE_SHIFT;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int64_t row = row_of[ty * 4 + r];
            if (row < 0) continue;
            const double v = bad ? nan : __dadd_rn(acc[r][c], comp[r][c]);
            double *out = C + row + j * ldc;
            const double t = __dmul_rn(alpha, v);
            *out = beta != 0.0 ? __dadd_rn(*out, t) : t;
        }
    }
}

}  // namespace

oz_status_t launch_native_rows(int64_t m, int64_t n, int64_t k, const double *A, int64_t lda,
                               const double *B, int64_t ldb, const int *list, const unsigned int *count,
                               const int32_t *shiftB, double alpha, double beta, double *C, int64_t ldc,
                               cudaStream_t stream)
{
    const int64_t gy = (m + kFbRows - 1) / kFbRows, gx = (n + kFbCols - 1) / kFbCols;
    if (gy > 65535 || gx > 2147483647ll) return OZ_ERR_UNSUPPORTED;
    dim3 grid(static_cast<unsigned>(gx), static_cast<unsigned>(gy));
    native_rows_kernel<<<grid, kFbThreads, 0, stream>>>(m, n, k, A, lda, B, ldb, list, count, shiftB, alpha, beta,
                                                       C, ldc);
    count_launch();
    OZ_CUDA_CHECK(cudaGetLastError());
    return OZ_OK;
}

}  // namespace oz
