// Reconstruction (Algorithm 3; Eq. 4-5 and the last step of Sec. 2 (iv)): residues -> the integer
// c' in [-M/2, M/2), unscaled by 2^-(sigma_i + tau_j) and rounded once to FP64.
//
// The paper's SIMT branch walks Garner's mixed-radix digits (r(r-1)/2 multiply-reduce steps).
// CRT fixes c' uniquely, so any exact evaluation gives the same integer; this kernel uses the
// weighted form
//     c' = sum_i c_i V_i  -  kappa M,     V_i = ((M/m_i)^-1 mod m_i) (M/m_i) mod M,
// with every V_i and M cut into three 38-bit chunks (40-bit for the all-byte set).  A stored
// residue is below 2 m_i < 2^11.1 (the whole-method calls keep a representative in (0, 2 m_i); 2^8
// for the byte set), so each of the three chunk sums is an integer below 2^53 -- at most 2^52.8 --
// and is formed EXACTLY by FP64 fused multiply-adds (r MACs per chunk).  kappa = round(S/M) comes from a floating estimate; the
// carry-normalised chunks are then summed with error-free additions, which give the correctly
// rounded FP64 value directly unless c' lies within a hair of a rounding boundary, of a power of
// two or of +-M/2 -- those rare outputs take an exact path: the 128-bit integer, an exact range
// test for the lift to [-M/2, M/2), and one round-to-nearest-even done in integer arithmetic.
// A thread handles the consecutive rows whose residues share one 32-bit word per modulus (two
// uint16, or four uint8 for the all-byte set).
#include <utility>

#include "oz_internal.h"

namespace oz {
namespace {

struct ReconConst {
    double V[kMaxR][3];        // V_i = V0 + V1 2^38 + V2 2^76
    double Mc[3];              // M   = M0 + M1 2^38 + M2 2^76
    double inv_M;              // 1/M (rounded)
    double half_M_guard;       // (M/2) (1 - 2^-30): beyond it the lift is decided exactly
    unsigned long long M_lo, M_hi;
};

__constant__ ReconConst c_recon[kNumSets];

// Chunk width: 38 bits for S and E (stored residues < 2^11.1, 13 terms: sums < 2^52.8); 40 bits for
// the 117.8-bit set A (residues < 2^8, 15 terms: sums < 2^52), so that three chunks cover M.
__host__ __device__ constexpr int chunk_bits(int set) { return set == 2 ? 40 : 38; }
__host__ __device__ constexpr double pow2d(int e) { double v = 1.0; for (int i = 0; i < e; ++i) v *= 2.0; return v; }
constexpr double kRint = 6755399441055744.0;          // 1.5 * 2^52: (x + kRint) - kRint = rint(x)

// x * 2^scale for a finite double x (exact unless the result leaves the normal range)
__device__ __forceinline__ double scale_pow2(double x, int scale)
{
    int hi = __double2hiint(x);
    int be = (hi >> 20) & 0x7FF;
    int nb = be + scale;
    if (be != 0 && nb >= 1 && nb <= 2046) return __hiloint2double(hi + (scale << 20), __double2loint(x));
    return scalbn(x, scale);        // zero, or a result outside the normal range
}

// w packs the residues of consecutive rows (two uint16 or four uint8); HALF selects the row
template <int SET, int HALF, int I>
__device__ __forceinline__ void crt_term(uint32_t w, double &S0, double &S1, double &S2)
{
    const ReconConst &K = c_recon[SET];
    constexpr int BITS = 8 * residue_bytes(SET);
    const uint32_t c = (w >> (BITS * HALF)) & ((1u << BITS) - 1u);
    // exact; the hardware conversion keeps this off the FP64 pipe, which bounds the kernel
    double cd = __uint2double_rn(c);
    S0 = fma(cd, K.V[I][0], S0);
    S1 = fma(cd, K.V[I][1], S1);
    S2 = fma(cd, K.V[I][2], S2);
}

template <int SET, int HALF, int... I>
__device__ __forceinline__ void crt_sum(std::integer_sequence<int, I...>, const uint32_t (&c)[kMaxR],
                                        double &S0, double &S1, double &S2)
{
    (crt_term<SET, HALF, I>(c[I], S0, S1, S2), ...);
}

// Exact tail (rare path): the normalised chunks as a 128-bit integer, exact lift to
// [-M/2, M/2), round-to-nearest-even conversion in integer arithmetic, power-of-two scale.
__device__ __noinline__ double finish_exact(double T0, double T1, double T2, int shift_sum, int set)
{
    const ReconConst &K = c_recon[set];
    const long long t0 = __double2ll_rn(T0), t1 = __double2ll_rn(T1), t2 = __double2ll_rn(T2);
    // v = t0 + t1 2^cw + t2 2^(2cw) as a two's-complement (hi:lo) pair
    const int cw = chunk_bits(set);
    unsigned long long lo = static_cast<unsigned long long>(t0) + (static_cast<unsigned long long>(t1) << cw);
    long long hi = (t0 >> 63) + (t1 >> (64 - cw)) + (lo < static_cast<unsigned long long>(t0) ? 1 : 0) +
                   static_cast<long long>(static_cast<unsigned long long>(t2) << (2 * cw - 64));
    const __int128 M = static_cast<__int128>((static_cast<unsigned __int128>(K.M_hi) << 64) | K.M_lo);
    const __int128 Mh = M >> 1;     // M is even for every set (each holds a power of two)
    __int128 v = static_cast<__int128>((static_cast<unsigned __int128>(static_cast<unsigned long long>(hi)) << 64) | lo);
    if (v >= Mh) v -= M;
    else if (v < -Mh) v += M;
    lo = static_cast<unsigned long long>(v);
    hi = static_cast<long long>(v >> 64);
    const bool neg = hi < 0;
    if (neg) {
        lo = 0ull - lo;
        hi = ~hi + (lo == 0ull ? 1 : 0);
    }
    // nearest double, ties to even: top 64 bits with a sticky bit far below the rounding position
    const unsigned long long uhi = static_cast<unsigned long long>(hi);
    const int lz = __clzll(static_cast<long long>(uhi | 1ull));          // uhi < 2^49: lz in [15, 63]
    const unsigned long long top = (uhi << lz) | (lo >> (64 - lz));
    const unsigned long long rest = lo << lz;
    unsigned long long mant = uhi ? (top | (rest ? 1ull : 0ull)) : lo;
    int scale = (uhi ? 64 - lz : 0) - shift_sum;
    double d = scale_pow2(__ull2double_rn(mant), scale);
    return neg ? -d : d;
}

template <int SET, int HALF>
__device__ __forceinline__ double reconstruct_one(const uint32_t (&c)[kMaxR], int shift_sum)
{
    const ReconConst &K = c_recon[SET];
    double S0 = 0.0, S1 = 0.0, S2 = 0.0;
    crt_sum<SET, HALF>(std::make_integer_sequence<int, set_r(SET)>{}, c, S0, S1, S2);
    constexpr double kTwo38 = pow2d(chunk_bits(SET));          // 2^cw  (names kept from the 38-bit case)
    constexpr double kTwoM38 = 1.0 / pow2d(chunk_bits(SET));   // 2^-cw
    constexpr double kTwo76 = kTwo38 * kTwo38;                 // 2^(2cw)
    double val = fma(S2, kTwo76, fma(S1, kTwo38, S0));
    double kappa = (val * K.inv_M + kRint) - kRint;
    double T0 = fma(-kappa, K.Mc[0], S0);              // exact: integers below 2^53
    double T1 = fma(-kappa, K.Mc[1], S1);
    double T2 = fma(-kappa, K.Mc[2], S2);
    // carry-normalise so that the three chunks do not overlap: |T0|, |T1| <= 2^37
    double c0 = (T0 * kTwoM38 + kRint) - kRint;
    T0 = fma(-c0, kTwo38, T0);
    T1 += c0;
    double c1 = (T1 * kTwoM38 + kRint) - kRint;
    T1 = fma(-c1, kTwo38, T1);
    T2 += c1;
    // c' = X2 + X1 + X0 exactly.  Fast path: two error-free additions give r = RN(s + t) and
    // the exact residual rem of that last rounding; r is the correctly rounded value of c'
    // unless c' lies within a hair of a rounding boundary (|rem| ~ half an ulp, or r a power
    // of two) or within a hair of +-M/2 (where the symmetric lift could apply).  Those cases,
    // a vanishing fraction of random data, take the exact integer path.
    const double X2 = T2 * kTwo76, X1 = T1 * kTwo38;   // exact
    const double s = X2 + X1;
    const double err = X1 - (s - X2);                   // exact: s + err = X2 + X1
    const double t = err + T0;
    const double r = s + t;
    const double rem = t - (r - s);                     // exact: r + rem = s + t
    const long long rb = __double_as_longlong(r);
    const int eb = static_cast<int>((rb >> 52) & 0x7FF);
    if (eb == 0) return 0.0;                            // c' = 0 (r is an integer: never subnormal)
    const double half_ulp = __longlong_as_double(static_cast<long long>(eb - 53) << 52);
    const bool near_tie = fabs(rem) >= fma(-half_ulp, 9.313225746154785e-10, half_ulp);   // (1 - 2^-30)
    const bool pow2 = (rb & 0xFFFFFFFFFFFFFll) == 0 && rem != 0.0;
    const bool near_half_M = fabs(r) >= K.half_M_guard;
    if (near_tie || pow2 || near_half_M) return finish_exact(T0, T1, T2, shift_sum, SET);
    return scale_pow2(r, -shift_sum);
}

// one row of the thread's group: reconstruct, scale by alpha
template <int SET, int H>
__device__ __forceinline__ double row_value(const uint32_t (&w)[kMaxR], int sa, int sb, double alpha)
{
    const double nan = __longlong_as_double(0x7FF8000000000000ll);
    double p = (sb == OZ_NONFINITE_SHIFT || sa == OZ_NONFINITE_SHIFT) ? nan : reconstruct_one<SET, H>(w, sa + sb);
    return p * alpha;
}

// scalar stores of up to two consecutive rows; `first` / `second`: which of them are written
__device__ __forceinline__ void store_pair(double *out, double p0, double p1, bool first, bool second, double beta)
{
    if (first) out[0] = beta != 0.0 ? out[0] + p0 : p0;
    if (second) out[1] = beta != 0.0 ? out[1] + p1 : p1;
}

// the ROWS consecutive rows of column j whose residues are packed in w[]: reconstruct, update C.
// For beta = 1 the old values of C are requested before the arithmetic starts, so that their latency
// hides behind it.  `keep`: bit h set = row h is written (rows that go to the native FP64 path are not).
template <int SET>
__device__ __forceinline__ void reconstruct_rows(const uint32_t (&w)[kMaxR], int64_t row, int nrows, int sb,
                                                 const int32_t *__restrict__ shiftA, double alpha, double beta,
                                                 double *out, bool vecC, uint32_t keep = 0xFu)
{
    constexpr int ROWS = 4 / residue_bytes(SET);
    int sa[ROWS];
#pragma unroll
    for (int h = 0; h < ROWS; ++h) sa[h] = h < nrows ? shiftA[row + h] : 0;
    const bool whole = vecC && nrows == ROWS && (keep & ((1u << ROWS) - 1u)) == ((1u << ROWS) - 1u);
    double2 old[ROWS / 2];
#pragma unroll
    for (int h = 0; h < ROWS / 2; ++h) old[h] = make_double2(0.0, 0.0);
    if (whole && beta != 0.0) {
#pragma unroll
        for (int h = 0; h < ROWS / 2; ++h) old[h] = *reinterpret_cast<const double2 *>(out + 2 * h);
    }
    {
        double p0 = row_value<SET, 0>(w, sa[0], sb, alpha);
        double p1 = nrows > 1 ? row_value<SET, 1>(w, sa[1], sb, alpha) : 0.0;
        if (whole) *reinterpret_cast<double2 *>(out) = make_double2(old[0].x + p0, old[0].y + p1);
        else store_pair(out, p0, p1, (keep & 1u) != 0, nrows > 1 && (keep & 2u) != 0, beta);
    }
    if constexpr (ROWS == 4) {
        if (nrows > 2) {
            double p2 = row_value<SET, 2>(w, sa[2], sb, alpha);
            double p3 = nrows > 3 ? row_value<SET, 3>(w, sa[3], sb, alpha) : 0.0;
            if (whole) *reinterpret_cast<double2 *>(out + 2) = make_double2(old[1].x + p2, old[1].y + p3);
            else store_pair(out + 2, p2, p3, (keep & 4u) != 0, nrows > 3 && (keep & 8u) != 0, beta);
        }
    }
}

// Each thread reconstructs ROWS consecutive rows of one column: the residues of those rows are one
// 32-bit word per modulus (two uint16 for S and E, four uint8 for the all-byte set A).
// Six blocks per SM (40 registers) for the two-byte sets: the kernel is bound by instruction issue
// and gains from the extra warps; the four-row variant of set A would spill at that budget.
template <int SET>
__global__ void __launch_bounds__(256, residue_bytes(SET) == 2 ? 6 : 5)
reconstruct_kernel(const void *__restrict__ Rv, int64_t ldr, int64_t mod_stride, int64_t m,
                   int64_t n, const int32_t *__restrict__ shiftA, const int32_t *__restrict__ shiftB,
                   double alpha, double beta, double *__restrict__ C, int64_t ldc, int vecR, int vecC)
{
    constexpr int RB = residue_bytes(SET), ROWS = 4 / RB, r = set_r(SET);
    // grid.x covers the row groups of a column, grid.y (and .z beyond 65535) the columns: no division
    const int64_t row = (blockIdx.x * 256ll + threadIdx.x) * ROWS;
    if (row >= m) return;
    const int64_t j = blockIdx.y + 65535ll * blockIdx.z;
    if (j >= n) return;
    const int nrows = m - row < ROWS ? static_cast<int>(m - row) : ROWS;

    // all residue loads are issued before any arithmetic: r independent requests in flight per
    // thread, kept packed so that they fit the register budget
    uint32_t w[kMaxR];
    const unsigned char *base = static_cast<const unsigned char *>(Rv) + (j * ldr + row) * RB;
#pragma unroll
    for (int i = 0; i < r; ++i) {
        const unsigned char *src = base + i * mod_stride * RB;
        if (vecR) {
            w[i] = *reinterpret_cast<const uint32_t *>(src);       // ldr is a multiple of ROWS: in bounds
        } else {
            uint32_t v = 0;
#pragma unroll
            for (int h = 0; h < ROWS; ++h) {
                if (h < nrows) {
                    uint32_t e = RB == 2 ? reinterpret_cast<const uint16_t *>(src)[h] : src[h];
                    v |= e << (8 * RB * h);
                }
            }
            w[i] = v;
        }
    }
    reconstruct_rows<SET>(w, row, nrows, shiftB[j], shiftA, alpha, beta, C + row + j * ldc, vecC != 0);
}

// Same reconstruction from the tile-ordered private array that the whole-method GEMM writes (see
// ResidueTiling).  A thread takes one 32-bit word of a 32-column x 64-row block, i.e. ROWS consecutive
// rows of one column.  The words of one column are dealt to consecutive threads, so that a warp
// reads and writes 512 contiguous bytes of C (one or two whole columns of the block); its residue
// loads are 16-byte pieces 512 bytes apart, and the warps of a thread block, which take neighbouring
// columns, ask for whole 128-byte lines between them.
// grid: x = (piece of the block, block within the tile, CTA rank of the pair), y = tile column, z = tile row
// SKIP: rows flagged in `skip` are left untouched (they are re-issued on the native FP64 path).
template <int SET, bool SKIP>
__global__ void __launch_bounds__(256, residue_bytes(SET) == 2 ? 6 : 5)
reconstruct_tiled_kernel(const void *__restrict__ Rv, int cg, int tiles_n, int tn0,
                         int64_t m, int64_t n, int64_t col0, int64_t col1,
                         const int32_t *__restrict__ shiftA, const int32_t *__restrict__ shiftB,
                         double alpha, double beta, double *__restrict__ C, int64_t ldc, int vecC,
                         const unsigned char *__restrict__ skip)
{
    constexpr int RB = residue_bytes(SET), ROWS = 4 / RB, r = set_r(SET);
    constexpr int kBlockWords = 64 * 32 * RB / 4;          // words of one 32 x 64 block: 1024 or 512
    constexpr int kColWords = 64 / ROWS;                   // words of one column of the block: 32 or 16
    constexpr int kCtaCols = 256 / kColWords;              // columns per thread block: 8 or 16
    constexpr int kPieces = 32 / kCtaCols;                 // thread blocks per residue block: 4 or 2
    const uint32_t piece = blockIdx.x % kPieces;
    const uint32_t wi = (blockIdx.x / kPieces) & 15u;
    const uint32_t rank = blockIdx.x / (kPieces * 16);     // 0, or 0..1 with CTA pairs
    const uint32_t tn = static_cast<uint32_t>(tn0) + blockIdx.y, tm = blockIdx.z;
    const uint32_t lane = piece * kCtaCols + threadIdx.x / kColWords;   // column of the block
    const uint32_t wq = threadIdx.x % kColWords, c = wq >> 2, sub = wq & 3u;
    const int64_t row = static_cast<int64_t>(tm) * 256 + (wi >> 2) * 64 + c * (16 / RB) + sub * ROWS;
    const int64_t j = (static_cast<int64_t>(tn) * cg + rank) * 128 + (wi & 3u) * 32 + lane;
    if (row >= m || j >= n || j < col0 || j >= col1) return;
    const int nrows = m - row < ROWS ? static_cast<int>(m - row) : ROWS;
    uint32_t keep = 0xFu;
    if constexpr (SKIP) {
        keep = 0u;
#pragma unroll
        for (int h = 0; h < ROWS; ++h)
            if (h < nrows && !skip[row + h]) keep |= 1u << h;
        if (!keep) return;
    }
    const int64_t wb = ((static_cast<int64_t>(tm) * tiles_n + tn) * cg + rank) * 16 + wi;
    // the r blocks of this patch are consecutive: modulus i at a compile-time offset
    const unsigned char *base = static_cast<const unsigned char *>(Rv) +
                                ((wb * r) * kBlockWords + c * 128 + lane * 4 + sub) * 4;
    uint32_t w[kMaxR];
#pragma unroll
    for (int i = 0; i < r; ++i) w[i] = *reinterpret_cast<const uint32_t *>(base + i * (kBlockWords * 4));
    reconstruct_rows<SET>(w, row, nrows, shiftB[j], shiftA, alpha, beta, C + row + j * ldc, vecC != 0, keep);
}

}  // namespace

oz_status_t upload_reconstruct_constants()
{
    static ReconConst host[kNumSets];
    for (int set = 0; set < kNumSets; ++set) {
        unsigned __int128 M = 1;
        for (int i = 0; i < set_r(set); ++i) M *= static_cast<unsigned>(modulus(set, i));
        const int cw = chunk_bits(set);
        const unsigned __int128 mask = (static_cast<unsigned __int128>(1) << cw) - 1;
        ReconConst &K = host[set];
        for (int i = 0; i < kMaxR; ++i) K.V[i][0] = K.V[i][1] = K.V[i][2] = 0.0;
        for (int i = 0; i < set_r(set); ++i) {
            unsigned mi = static_cast<unsigned>(modulus(set, i));
            unsigned __int128 W = M / mi;
            unsigned wm = static_cast<unsigned>(W % mi), inv = 0;
            for (unsigned c = 1; c < mi; ++c)
                if ((static_cast<unsigned long long>(wm) * c) % mi == 1) { inv = c; break; }
            unsigned __int128 V = W * inv;          // < M, and V = 1 mod m_i, 0 mod the other moduli
            K.V[i][0] = static_cast<double>(static_cast<unsigned long long>(V & mask));
            K.V[i][1] = static_cast<double>(static_cast<unsigned long long>((V >> cw) & mask));
            K.V[i][2] = static_cast<double>(static_cast<unsigned long long>(V >> (2 * cw)));
        }
        K.Mc[0] = static_cast<double>(static_cast<unsigned long long>(M & mask));
        K.Mc[1] = static_cast<double>(static_cast<unsigned long long>((M >> cw) & mask));
        K.Mc[2] = static_cast<double>(static_cast<unsigned long long>(M >> (2 * cw)));
        K.inv_M = 1.0 / static_cast<double>(M);
        K.half_M_guard = 0.5 * static_cast<double>(M) * (1.0 - 9.313225746154785e-10);
        K.M_lo = static_cast<unsigned long long>(M);
        K.M_hi = static_cast<unsigned long long>(M >> 64);
    }
    OZ_CUDA_CHECK(cudaMemcpyToSymbol(c_recon, host, sizeof(host)));
    return OZ_OK;
}

oz_status_t launch_reconstruct(int64_t m, int64_t n, const void *R, int64_t ldr,
                               int64_t mod_stride, const int32_t *shiftA, const int32_t *shiftB,
                               int set, double alpha, double beta, double *C, int64_t ldc,
                               cudaStream_t stream)
{
    // one 32-bit load per modulus covers a thread's rows when every row group starts on a 4-byte boundary
    const int rows = 4 / residue_bytes(set);
    int vecR = (ldr % rows == 0 && mod_stride % rows == 0 && (reinterpret_cast<uintptr_t>(R) & 3u) == 0) ? 1 : 0;
    int vecC = ((ldc & 1) == 0 && (reinterpret_cast<uintptr_t>(C) & 15u) == 0) ? 1 : 0;
    int64_t bx = ((m + rows - 1) / rows + 255) / 256;
    if (bx > 0x7FFFFFFFll) return OZ_ERR_UNSUPPORTED;
    if (n > 65535ll * 65535ll) return OZ_ERR_UNSUPPORTED;
    dim3 grid(static_cast<unsigned>(bx), static_cast<unsigned>(n < 65535 ? n : 65535),
              static_cast<unsigned>((n + 65534) / 65535));
    if (set == 2)
        reconstruct_kernel<2><<<grid, 256, 0, stream>>>(R, ldr, mod_stride, m, n, shiftA, shiftB, alpha,
                                                        beta, C, ldc, vecR, vecC);
    else if (set == 0)
        reconstruct_kernel<0><<<grid, 256, 0, stream>>>(R, ldr, mod_stride, m, n, shiftA, shiftB, alpha,
                                                        beta, C, ldc, vecR, vecC);
    else
        reconstruct_kernel<1><<<grid, 256, 0, stream>>>(R, ldr, mod_stride, m, n, shiftA, shiftB, alpha,
                                                        beta, C, ldc, vecR, vecC);
    count_launch();
    OZ_CUDA_CHECK(cudaGetLastError());
    return OZ_OK;
}

oz_status_t launch_reconstruct_tiled(int64_t m, int64_t n, const void *R, const int32_t *shiftA,
                                     const int32_t *shiftB, int set, double alpha, double beta,
                                     double *C, int64_t ldc, int64_t col0, int64_t col1,
                                     cudaStream_t stream, const unsigned char *skip)
{
    if (col1 <= col0) return OZ_OK;
    const ResidueTiling t = residue_tiling(m, n, set);
    const int tn0 = static_cast<int>(col0 / t.tile_cols);
    const int ntn = static_cast<int>((col1 + t.tile_cols - 1) / t.tile_cols) - tn0;
    const int pieces = 64 * 32 * residue_bytes(set) / 4 / 256;
    if (t.tiles_m > 65535 || ntn > 65535) return OZ_ERR_UNSUPPORTED;
    const int vecC = ((ldc & 1) == 0 && (reinterpret_cast<uintptr_t>(C) & 15u) == 0) ? 1 : 0;
    const dim3 grid(static_cast<unsigned>(pieces * 16 * t.cg), static_cast<unsigned>(ntn),
                    static_cast<unsigned>(t.tiles_m));
#define OZ_RECON_TILED(SET_)                                                                               \
    (skip ? reconstruct_tiled_kernel<SET_, true><<<grid, 256, 0, stream>>>(                                \
                R, t.cg, t.tiles_n, tn0, m, n, col0, col1, shiftA, shiftB, alpha, beta, C, ldc, vecC, skip) \
          : reconstruct_tiled_kernel<SET_, false><<<grid, 256, 0, stream>>>(                               \
                R, t.cg, t.tiles_n, tn0, m, n, col0, col1, shiftA, shiftB, alpha, beta, C, ldc, vecC, nullptr))
    if (set == 2) OZ_RECON_TILED(2);
    else if (set == 0) OZ_RECON_TILED(0);
    else OZ_RECON_TILED(1);
#undef OZ_RECON_TILED
    count_launch();
    OZ_CUDA_CHECK(cudaGetLastError());
    return OZ_OK;
}

}  // namespace oz
