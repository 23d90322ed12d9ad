// Internal declarations shared by the translation units of liboz_b200.so.
// Nothing here is part of the public ABI (see include/oz.h).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "oz.h"

namespace oz {

constexpr int kMaxR = 15;          // moduli in the largest supported set (A)
constexpr int kMaxPlanes = 44;     // stored planes of set A with two-limb digits
// The plane look-up table of a set holds, per modulus, the packed plane bytes of the residues 0 .. m-1.
constexpr int kLutSpan = 1;
constexpr int kLutWords = 8208;    // >= sum of the moduli of any set (S: 8069, E: 6736, A: 3478)

// ---- modulus sets (Sec. 2 step (ii) for S; "Candidate E" and "Candidate A" paragraphs) ---
constexpr int kNumSets = 3;
__host__ __device__ constexpr int set_r(int set) { return set == 0 ? 12 : (set == 1 ? 13 : 15); }

__host__ __device__ constexpr int modulus(int set, int i)
{
    constexpr int S[15] = {1089, 1024, 961, 841, 625, 529, 511, 509, 503, 499, 491, 487, 1, 1, 1};
    constexpr int E[15] = {1089, 1024, 961, 841, 625, 529, 251, 247, 241, 239, 233, 229, 227, 1, 1};
    constexpr int A[15] = {256, 255, 253, 251, 247, 241, 239, 233, 229, 227, 223, 217, 211, 199, 197};
    return set == 0 ? S[i] : (set == 1 ? E[i] : A[i]);
}

// bytes of one stored residue in [0, m): the moduli of set A fit a byte
__host__ __device__ constexpr int residue_bytes(int set) { return set == 2 ? 1 : 2; }

// square root of a square modulus, 0 otherwise
__host__ __device__ constexpr int square_root(int m)
{
    for (int s = 2; s * s <= m; ++s)
        if (s * s == m) return s;
    return 0;
}

// Plane layouts of one operand:
//   kLayoutDigits  2 (square) or 3 digit planes per modulus: d0, d1[, d0+d1]   (Sec. 2 "FP8 variant")
//   kLayoutNative  1 plane: the centred residue itself as an INT8 operand (byte moduli only;
//                  Sec. 2 "The substrate transition")
//   kLayoutMerged  the A operand of the merged-accumulator schedule (discussion of Table "tuples",
//                  N_acc = 2): the d1 plane of every non-square modulus holds the pre-scaled -16*d1
//                  (d1 enters only through d1*e1); same plane count as kLayoutDigits
//   kLayoutMergedI8A / kLayoutMergedI8B  the same schedule on INT8 digit planes, where -16*d1 does
//                  not fit a byte: both operands carry 4*d1 in place of d1 and the A operand -d0
//                  in place of d0, so that (-d0) e0 + (4 d1)(4 e1) = -(d0 e0 - 16 d1 e1)
constexpr int kLayoutDigits = 0, kLayoutNative = 1, kLayoutMerged = 2, kLayoutMergedI8A = 3,
              kLayoutMergedI8B = 4;

__host__ __device__ constexpr int planes_of(int m, int layout = kLayoutDigits)
{
    return layout == kLayoutNative ? 1 : (square_root(m) ? 2 : 3);
}

__host__ __device__ constexpr int first_plane(int set, int i, int layout = kLayoutDigits)
{
    int p = 0;
    for (int j = 0; j < i; ++j) p += planes_of(modulus(set, j), layout);
    return p;
}

__host__ __device__ constexpr int p_store(int set, int layout = kLayoutDigits)
{
    return first_plane(set, set_r(set), layout);
}

// largest k for which the merged accumulator d0 e0 - 16 d1 e1 stays exact in FP32: the merged term
// reaches 4095 on the 9-bit tail of S and 1088 on byte moduli
__host__ __device__ constexpr int64_t merged_k_limit(int set) { return set == 0 ? 4097 : 15420; }

__host__ __device__ constexpr int lut_offset(int set, int i)
{
    int o = 0;
    for (int j = 0; j < i; ++j) o += kLutSpan * modulus(set, j);
    return o;
}

// words of a set's table, rounded up to whole 16-byte groups
__host__ __device__ constexpr int lut_words(int set) { return (lut_offset(set, set_r(set)) + 3) / 4 * 4; }

// 2^e mod m
__host__ __device__ constexpr uint32_t pow2_mod(int e, uint32_t m)
{
    uint32_t v = 1 % m;
    for (int j = 0; j < e; ++j) v = (v * 2u) % m;
    return v;
}

// smallest s with 2^s >= m
__host__ __device__ constexpr int ceil_log2(uint32_t m)
{
    int s = 0;
    while ((1u << s) < m) ++s;
    return s;
}

// floor(2^32 / m)
__host__ __device__ constexpr uint32_t barrett_magic(uint32_t m)
{
    return static_cast<uint32_t>(0x100000000ull / m);
}

inline int64_t round_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }

// ---- route decoding ----------------------------------------------------------------------
struct Route {
    int substrate;  // 0 fp8, 1 int8 (two-limb digits), 2 int8 native (one residue plane, set A only)
    int acc;        // 0 unspecified, 1 merged accumulators, 2 separate accumulators
    bool native() const { return substrate == 2; }
    bool merged() const { return acc == 1; }
    // plane layout of the operand on `side` (0: rows of A, 1: columns of B)
    int layout(int side) const
    {
        if (native()) return kLayoutNative;
        if (!merged()) return kLayoutDigits;
        if (substrate == 1) return side == 0 ? kLayoutMergedI8A : kLayoutMergedI8B;
        return side == 0 ? kLayoutMerged : kLayoutDigits;
    }
    bool hosted;    // whole-method calls: CRT recombination on the INT8 tensor pipe (OZ_RECON_TENSOR)
    bool fallback;  // oz_dgemm / oz_dgemm_ex: out-of-range rows re-issued on the native FP64 path
    bool fused;     // oz_dgemm / oz_dgemm_ex: A converted inside the product kernel (storage mode F)
    int quant;      // 0 rn, 1 tz
    int rule;       // 0 maxexp, 1 cs, 2 accurate (shifts from the extra bound product)
};
bool decode_route(uint32_t route, Route *out);
bool decode_route_for_set(int set, uint32_t route, Route *out);
oz_status_t resolve_schedule(int set, int64_t k, int64_t n, bool automatic, Route *rt);   // merged or separate accumulators   // also rejects native INT8 off set A

// ---- per-device state --------------------------------------------------------------------
// Builds the lookup tables and constant blocks on the current device the first time it is used.
oz_status_t ensure_device_ready();

// device addresses of the per-device objects (valid after ensure_device_ready())
const uint32_t *device_lut(int set, int substrate);  // kLutWords packed plane bytes
unsigned int *device_status_word();

void count_launch(int n = 1);

// quantisation budgets (host)
void budget_maxexp(int set, int64_t k, int *tA, int *tB);
void cs_bound_squared(int set, int64_t k, uint64_t *lo, uint64_t *hi);  // G^2 as 128 bits

// ---- stage launchers (host side of each .cu) ---------------------------------------------
oz_status_t launch_deconstruct(int side, int64_t lines, int64_t k, const double *X, int64_t ldx,
                               int set, const Route &rt, uint8_t *planes, int64_t plane_stride,
                               int64_t row_pitch, int32_t *shift, void *scratch,
                               cudaStream_t stream);

// Tile-ordered private residue array of the whole-method calls.  The output is cut into tiles of
// 256 rows x tile_cols columns (128, or 256 when CTA pairs are used); a tile is 16 blocks (32 with
// pairs: rank-major) of 32 columns x 64 rows, one per epilogue warp, block w = quarter + 4 * part
// covering columns 32 * quarter .. +31 (of the rank's 128) and rows 64 * part .. +63; a block is
// stored as [16-byte chunk c][column], chunk c holding 16 / residue_bytes consecutive rows.
// Order in memory: tile row, tile column, CTA rank, block, modulus -- the r residue blocks of one
// 32 x 64 patch of the output are consecutive (4 KiB each, 2 KiB for byte residues).
struct ResidueTiling {
    int cg;              // 1: tiles of 128 columns, 2: CTA pairs, tiles of 256 columns
    int tile_cols;
    int tiles_m, tiles_n;
    int64_t mod_stride;  // elements per modulus in total (tiles are stored whole, padding included)
};
ResidueTiling residue_tiling(int64_t m, int64_t n, int set);

// loose: residues in [0, 2 m_i) (two-byte sets); tiled: R is the tile-ordered private array
// (ldr and mod_stride are then ignored)
// pieces of launch_deconstruct, and the steps of the accurate rule between them
oz_status_t launch_scan(int side, int64_t lines, int64_t k, const double *X, int64_t ldx, int set,
                        const Route &rt, int32_t *shift, void *scratch, cudaStream_t stream);
oz_status_t launch_convert_planes(int side, int64_t lines, int64_t k, const double *X, int64_t ldx,
                                  int set, const Route &rt, uint8_t *planes, int64_t plane_stride,
                                  int64_t row_pitch, const int32_t *shift, cudaStream_t stream);
oz_status_t launch_bound_plane(int side, int64_t lines, int64_t k, const double *X, int64_t ldx,
                               void *scratch, uint8_t *plane, int64_t pitch, cudaStream_t stream);
unsigned int *bound_maxima(void *scratch, int64_t lines);      // one word per line, word stride 2
oz_status_t launch_accurate_finalize(int64_t lines, void *scratch, int budget_log2, int32_t *shift,
                                     cudaStream_t stream);
oz_status_t upload_bound_codes(const unsigned char *codes33);
// the bound product on the tensor cores: rowmax[2 i] / colmax[2 j] receive (atomicMax) the bit pattern
// of max_j / max_i of sum_k GA[i][k] GB[j][k], an integer-valued FP32 number; k <= kBoundKMax
constexpr int64_t kBoundKMax = 16384;
oz_status_t launch_bound_gemm(int64_t m, int64_t n, int64_t k, const uint8_t *GA, int64_t pitchA,
                              const uint8_t *GB, int64_t pitchB, unsigned int *rowmax,
                              unsigned int *colmax, cudaStream_t stream);
int accurate_budget_log2(int set);
// exponent-span check: threshold of the set against the product of the two operands' flatness codes
unsigned int esc_threshold(int set);

oz_status_t launch_residue_gemm(int64_t m, int64_t n, int64_t k, const uint8_t *PA,
                                int64_t strideA, int64_t pitchA, const uint8_t *PB,
                                int64_t strideB, int64_t pitchB, int set, const Route &rt,
                                void *R, int64_t ldr, int64_t mod_stride, bool loose, bool tiled,
                                cudaStream_t stream);

// Storage mode F: residue products with A converted on the fly inside the kernel (n <= 128, merged
// schedule on digit planes, k within the exact depth of one accumulator); public residue layout
bool fused_gemm_applies(int64_t m, int64_t n, int64_t k, int set, const Route &rt);
oz_status_t launch_fused_gemm(int64_t m, int64_t n, int64_t k, const double *A, int64_t lda, const int32_t *shiftA,
                              const uint8_t *PB, int64_t strideB, int64_t pitchB, int set, const Route &rt,
                              void *R, int64_t ldr, int64_t mod_stride, cudaStream_t stream);

// reconstruction from the tile-ordered array, columns [col0, col1) of the m x n output
oz_status_t launch_reconstruct_tiled(int64_t m, int64_t n, const void *R, const int32_t *shiftA,
                                     const int32_t *shiftB, int set, double alpha, double beta,
                                     double *C, int64_t ldc, int64_t col0, int64_t col1,
                                     cudaStream_t stream, const unsigned char *skip_rows = nullptr);

oz_status_t launch_reconstruct(int64_t m, int64_t n, const void *R, int64_t ldr,
                               int64_t mod_stride, const int32_t *shiftA, const int32_t *shiftB,
                               int set, double alpha, double beta, double *C, int64_t ldc,
                               cudaStream_t stream);

// uploads the reconstruction constants of every set to the current device
oz_status_t upload_reconstruct_constants();
oz_status_t upload_hosted_constants();

// reconstruction from the tile-ordered array with the CRT recombination on the INT8 tensor pipe
oz_status_t launch_reconstruct_hosted(int64_t m, int64_t n, const void *R, const int32_t *shiftA,
                                      const int32_t *shiftB, int set, double alpha, double beta,
                                      double *C, int64_t ldc, int64_t col0, int64_t col1,
                                      cudaStream_t stream);

// Out-of-range rows (Algorithm 1, last line; Algorithm 3, "ESC range check"): flags, ascending list and
// number of the rows that go to the native FP64 path, from the scan results that the three-pass
// deconstruction left in the two scratch blocks; and the native path itself
oz_status_t launch_esc_rows(void *scratchA, int64_t m, void *scratchB, int64_t n, int64_t k, int set,
                            unsigned char *flag, int *list, unsigned int *count, cudaStream_t stream);
oz_status_t launch_native_rows(int64_t m, int64_t n, int64_t k, const double *A, int64_t lda,
                               const double *B, int64_t ldb, const int *list, const unsigned int *count,
                               const int32_t *shiftB, double alpha, double beta, double *C, int64_t ldc,
                               cudaStream_t stream);

#define OZ_CUDA_CHECK(expr)                                  \
    do {                                                     \
        cudaError_t e__ = (expr);                            \
        if (e__ != cudaSuccess) return OZ_ERR_CUDA;          \
    } while (0)

}  // namespace oz
