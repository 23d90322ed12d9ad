// Deconstruction (Algorithm 2; scaling of Eq. 1): FP64 operand -> per-line shifts and K-major
// 8-bit residue planes.
//
// Kernels, in launch order for one operand:
//   scan_init      clears the per-line scratch (largest exponent, non-finite flag, sum of squares)
//   scan_maxexp    largest floor(log2|x|) of every line, Inf/NaN detection
//   scan_sumsq     CS rule only: exact integer sum of ceil(|x| 2^(9-E))^2 per line
//   scan_finalize  shift[line] (sigma_i or tau_j of Eq. 1)
//   convert        quantise, reduce modulo every modulus, look the plane bytes up, store
//
// The scan is split over the inner dimension with integer atomics (max / or / add), so its
// result does not depend on the order of the partial results: the shifts are bit-reproducible.
//
// Residue of a 64-bit two's-complement integer a' modulo m (the paper's byte-plane identity of
// paragraph "O2", applied to 16-bit limbs so that every partial sum stays below 2^32):
//   a' mod m = (l0 + l1 (2^16 mod m) + l2 (2^32 mod m) + l3 (2^48 mod m) + bias_m) mod m
// with the top limb l3 taken SIGNED (this replaces the paper's (-2^64) mod m sign correction) and
// bias_m a multiple of m that keeps the sum non-negative, followed by one exact multiply-high
// division by m.  The digit split, the Lemma 1 carry and the
// E4M3 / INT8 encoding are folded into a per-modulus table indexed by the canonical residue
// (built on the host at set-up), held in shared memory.
#include <utility>

#include "oz_internal.h"
#include "oz_convert.cuh"

namespace oz {
namespace {

constexpr int kConvThreads = 256;
constexpr int kChunk = 128;            // inner-dimension bytes handled per warp step (4 per lane)
constexpr int kTileLines = 32;         // side 0: lines per shared-memory transposition tile
constexpr int kTilePitch = kChunk + 1; // doubles per tile row (+1: conflict-free column writes)

struct ScanScratch {
    unsigned long long *sumsq;  // [lines]  sum of squared magnitudes (accurate rule: maximum of the bound product)
    int *emax;                  // [lines]  largest exponent, INT32_MIN for a line of zeros
    int *nonfinite;             // [lines]  bit 31: the line holds Inf/NaN; bits 0..30: sum of the magnitudes
};
constexpr int kNonfiniteBit = INT32_MIN;

__host__ __device__ inline ScanScratch carve_scratch(void *scratch, int64_t lines)
{
    ScanScratch s;
    char *base = static_cast<char *>(scratch);
    s.sumsq = reinterpret_cast<unsigned long long *>(base);
    s.emax = reinterpret_cast<int *>(base + 8 * lines);
    s.nonfinite = reinterpret_cast<int *>(base + 12 * lines);
    return s;
}

__device__ __forceinline__ const double *element(const double *X, int64_t ldx, int side,
                                                 int64_t line, int64_t kk)
{
    return side == 0 ? X + line + kk * ldx : X + kk + line * ldx;
}

// classification of a double: returns 0 zero, 1 finite non-zero (e = floor(log2|x|)), 2 Inf/NaN
__device__ __forceinline__ int classify(double x, int *e)
{
    unsigned long long bits = static_cast<unsigned long long>(__double_as_longlong(x));
    int be = static_cast<int>((bits >> 52) & 0x7FF);
    unsigned long long frac = bits & 0xFFFFFFFFFFFFFull;
    if (be == 0x7FF) return 2;
    if (be == 0) {
        if (frac == 0) return 0;
        *e = -1011 - __clzll(static_cast<long long>(frac));   // subnormal: normalise the fraction
        return 1;
    }
    *e = be - 1023;
    return 1;
}

__global__ void scan_init_kernel(ScanScratch s, int64_t lines)
{
    int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x;
    if (i < lines) {
        s.sumsq[i] = 0ull;
        s.emax[i] = INT32_MIN;
        s.nonfinite[i] = 0;
    }
}

// One pass over the operand.  PASS 0: largest exponent + non-finite flag.  PASS 1: sum of squares.
// side 0: thread = line, loop over a k-range (loads coalesced across lines).
// side 1: warp = line, lanes stride over a k-range (loads coalesced along k), shuffle reduction.
template <int SIDE, int PASS>
__global__ void __launch_bounds__(256)
scan_kernel(const double *__restrict__ X, int64_t ldx, int64_t lines, int64_t k, int64_t kspan,
            ScanScratch s)
{
    int64_t k0 = static_cast<int64_t>(blockIdx.y) * kspan;
    int64_t k1 = k0 + kspan < k ? k0 + kspan : k;
    int lane = threadIdx.x & 31;
    int64_t line;
    int64_t kstart, kstep;
    if (SIDE == 0) {
        line = blockIdx.x * 256ll + threadIdx.x;
        kstart = k0;
        kstep = 1;
    } else {
        line = blockIdx.x * 8ll + (threadIdx.x >> 5);
        kstart = k0 + lane;
        kstep = 32;
    }
    bool live = line < lines;
    int emax = INT32_MIN, bad = 0;
    unsigned long long acc = 0;
    unsigned int l1 = 0;          // sum of the magnitudes abar <= 2^10 (exponent-span check): below 2^30 for k <= 2^20
    int E = 0;
    if (PASS == 1 && live) E = s.emax[line];
    // 2^(9-E) as a double, when it is a normal number (not for lines of subnormals only)
    const bool fast_scale = PASS == 1 && E != INT32_MIN && 9 - E >= -1000 && 9 - E <= 1000;
    const double scale9 = __hiloint2double((1023 + (fast_scale ? 9 - E : 0)) << 20, 0);
    if (live && !(PASS == 1 && E == INT32_MIN)) {
        // batches of 8 independent loads keep enough bytes in flight to run at memory speed
        for (int64_t kb = kstart; kb < k1; kb += 8 * kstep) {
            double xs[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                int64_t kk = kb + u * kstep;
                xs[u] = kk < k1 ? *element(X, ldx, SIDE, line, kk) : 0.0;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                double x = xs[u];
                if (PASS == 0) {
                    int e;
                    int c = classify(x, &e);
                    if (c == 2) bad = 1;
                    if (c == 1 && e > emax) emax = e;
                } else if (fast_scale) {
                    // ceil(|x| 2^(9-E)) through an exact FP64 scaling and a round-up conversion; a
                    // non-zero x whose scaled value underflows to zero still counts as 1
                    double y = fabs(x) * scale9;
                    unsigned long long abar = static_cast<unsigned long long>(__double2ll_ru(y));
                    if (abar == 0ull && x != 0.0) abar = 1ull;
                    if (!(y < 2048.0)) abar = 0ull;       // Inf/NaN: the line is flagged, value unused
                    acc += abar * abar;
                    l1 += static_cast<unsigned int>(abar);
                } else {
                    unsigned long long bits = static_cast<unsigned long long>(__double_as_longlong(x));
                    int be = static_cast<int>((bits >> 52) & 0x7FF);
                    unsigned long long frac = bits & 0xFFFFFFFFFFFFFull;
                    if (be == 0x7FF || (be == 0 && frac == 0)) continue;
                    unsigned long long sig = be ? (frac | (1ull << 52)) : frac;
                    int ex = be ? be - 1023 : -1022;
                    int sh = 43 + E - ex;                 // |x| 2^(9-E) = sig / 2^sh
                    unsigned long long abar;
                    if (sh >= 64) abar = 1;
                    else if (sh <= 0) abar = sig << (-sh);
                    else abar = (sig >> sh) + ((sig & ((1ull << sh) - 1)) ? 1ull : 0ull);
                    acc += abar * abar;
                    l1 += static_cast<unsigned int>(abar);
                }
            }
        }
    }
    if (SIDE == 1) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            if (PASS == 0) {
                int other = __shfl_xor_sync(0xFFFFFFFFu, emax, o);
                emax = other > emax ? other : emax;
                bad |= __shfl_xor_sync(0xFFFFFFFFu, bad, o);
            } else {
                acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
                l1 += __shfl_xor_sync(0xFFFFFFFFu, l1, o);
            }
        }
        if (lane != 0) live = false;
    }
    if (!live) return;
    if (PASS == 0) {
        if (emax != INT32_MIN) atomicMax(&s.emax[line], emax);
        if (bad) atomicOr(&s.nonfinite[line], kNonfiniteBit);
    } else if (acc) {
        atomicAdd(&s.sumsq[line], acc);
        atomicAdd(&s.nonfinite[line], static_cast<int>(l1));     // never reaches bit 31
    }
}

// shift[line]: MAXEXP  t - 1 - E;  CS  p + 9 - E with p the largest integer such that
// 4^p * S <= G^2  (G^2 passed as two 64-bit words).
__global__ void scan_finalize_kernel(ScanScratch s, int64_t lines, int64_t k, int side, int rule, int tbits,
                                     unsigned long long g2lo, unsigned long long g2hi,
                                     unsigned int esc_threshold, int32_t *shift, unsigned int *status)
{
    int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x;
    if (i >= lines) return;
    if (s.nonfinite[i] < 0) {
        shift[i] = OZ_NONFINITE_SHIFT;
        atomicOr(status, 1u << OZ_ERR_NONFINITE_INPUT);
        return;
    }
    int E = s.emax[i];
    if (E == INT32_MIN) { shift[i] = 0; return; }
    if (rule == 0) { shift[i] = tbits - 1 - E; return; }
    unsigned __int128 G2 = (static_cast<unsigned __int128>(g2hi) << 64) | g2lo;
    unsigned __int128 q = G2 / static_cast<unsigned __int128>(s.sumsq[i]);   // >= 4^p  <=>  4^p S <= G^2
    unsigned long long qhi = static_cast<unsigned long long>(q >> 64);
    unsigned long long qlo = static_cast<unsigned long long>(q);
    int top = qhi ? 127 - __clzll(static_cast<long long>(qhi)) : 63 - __clzll(static_cast<long long>(qlo));
    shift[i] = (top >> 1) + 9 - E;
    // Exponent-span check (Algorithm 1, "ESC check"): flatness of the line,
    // floor(2^16 (sum abar)^2 / (k sum abar^2)); the smallest value of each operand is kept in the
    // device status block and judged against the set's threshold when the status is queried.
    const unsigned long long l1 = static_cast<unsigned int>(s.nonfinite[i]);
    const unsigned __int128 flat = ((static_cast<unsigned __int128>(l1 * l1)) << 16) /
                                   (static_cast<unsigned __int128>(static_cast<unsigned long long>(k)) * s.sumsq[i]);
    atomicMin(status + 1 + side, static_cast<unsigned int>(flat));
    status[3] = esc_threshold;
}

// ---- out-of-range rows (Algorithm 1, last line; Algorithm 3, "ESC range check; re-issue out-of-range
// rows on the native-FP64 path") ------------------------------------------------------------------
// flatness of one scanned line from its norm sums, capped at 2^16; 0xFFFFFFFF for a line that does
// not count (zeros only, or Inf/NaN)
__device__ __forceinline__ unsigned int scanned_flatness(const ScanScratch &s, int64_t i, int64_t k)
{
    const int nf = s.nonfinite[i];
    if (nf < 0 || s.emax[i] == INT32_MIN) return 0xFFFFFFFFu;
    const unsigned long long l1 = static_cast<unsigned int>(nf);
    const unsigned __int128 flat = ((static_cast<unsigned __int128>(l1 * l1)) << 16) /
                                   (static_cast<unsigned __int128>(static_cast<unsigned long long>(k)) * s.sumsq[i]);
    const unsigned int q = static_cast<unsigned int>(flat);
    return q > 65536u ? 65536u : q;
}

// One block.  Row i of the product is re-issued when q(a_i) * min_j q(b_j) < threshold.  Writes the
// flag of every row, the re-issued rows in ascending order, their number, and adds that number to the
// device status block (word 4).
__global__ void __launch_bounds__(1024)
esc_rows_kernel(ScanScratch sA, int64_t m, ScanScratch sB, int64_t n, int64_t k, unsigned int threshold,
                unsigned char *flag, int *list, unsigned int *count, unsigned int *status)
{
    __shared__ unsigned int red[32];
    __shared__ unsigned int base;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned int qb = 0xFFFFFFFFu;
    for (int64_t j = tid; j < n; j += blockDim.x) qb = min(qb, scanned_flatness(sB, j, k));
    qb = __reduce_min_sync(0xFFFFFFFFu, qb);
    if (lane == 0) red[warp] = qb;
    if (tid == 0) base = 0u;
    __syncthreads();
    qb = red[lane];
    qb = __reduce_min_sync(0xFFFFFFFFu, qb);
    if (qb > 65536u) qb = 65536u;
    __syncthreads();
    for (int64_t i0 = 0; i0 < m; i0 += blockDim.x) {
        const int64_t i = i0 + tid;
        bool out = false;
        if (i < m) {
            const unsigned int qa = scanned_flatness(sA, i, k);
            out = qa != 0xFFFFFFFFu && static_cast<unsigned long long>(qa) * qb < threshold;
            flag[i] = out ? 1 : 0;
        }
        // ordered compaction: position = rows re-issued so far + those of lower threads
        const unsigned int ballot = __ballot_sync(0xFFFFFFFFu, out);
        if (lane == 0) red[warp] = __popc(ballot);
        __syncthreads();
        unsigned int before = base;
        for (int w = 0; w < warp; ++w) before += red[w];
        if (out) list[before + __popc(ballot & ((1u << lane) - 1u))] = static_cast<int>(i);
        __syncthreads();
        if (tid == 0) {
            unsigned int total = 0;
            for (int w = 0; w < 32; ++w) total += red[w];
            base += total;
        }
        __syncthreads();
    }
    if (tid == 0) {
        *count = base;
        if (base) atomicAdd(status + 4, base);
    }
}

// ---- accurate mode (Sec. 2 "The FP8 variant": the additional FP8 product that estimates a
// magnitude bound, the "+1" of the 3r + 1 schedule) ------------------------------------------
// Magnitude digit of one element: the smallest integer of the E4M3 grid {0..16, 18, 20, .., 32} that
// is >= |x| 2^(4-E), E the largest exponent of the line; integer arithmetic on the bit pattern.
__device__ __forceinline__ uint32_t bound_digit(double x, int E)
{
    unsigned long long bits = static_cast<unsigned long long>(__double_as_longlong(x));
    int be = static_cast<int>((bits >> 52) & 0x7FF);
    unsigned long long frac = bits & 0xFFFFFFFFFFFFFull;
    if (be == 0x7FF || (be == 0 && frac == 0)) return 0u;
    unsigned long long sig = be ? (frac | (1ull << 52)) : frac;
    int ex = be ? be - 1023 : -1022;
    int sh = 48 + E - ex;                                 // |x| 2^(4-E) = sig / 2^sh
    unsigned long long g;
    if (sh >= 64) g = 1ull;
    else if (sh <= 0) g = sig << (-sh);
    else g = (sig >> sh) + ((sig & ((1ull << sh) - 1ull)) ? 1ull : 0ull);
    uint32_t d = static_cast<uint32_t>(g);
    if (d > 16u && (d & 1u)) ++d;                         // above 16 the grid holds the even integers
    return d;
}

__constant__ unsigned char c_bound_code[33];              // E4M3 byte of the digits 0..32

// One byte per element: the E4M3 code of its magnitude digit, K-major like the residue planes
// (out[line * pitch + kk]; bytes kk in [k, pitch) are zero).  Lines of zeros and lines with
// Inf/NaN give zeros.  SIDE 0 goes through a 32 x 32 shared-memory tile so that loads run along
// the lines and stores along k.
template <int SIDE>
__global__ void __launch_bounds__(256)
bound_plane_kernel(const double *__restrict__ X, int64_t ldx, int64_t lines, int64_t k, ScanScratch s,
                   uint8_t *__restrict__ out, int64_t pitch)
{
    __shared__ unsigned char tile[32][36];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;      // 32 x 8
    const int64_t kchunks = (pitch + 31) / 32;
    const int64_t ltiles = (lines + 31) / 32;
    for (int64_t item = blockIdx.x; item < ltiles * kchunks; item += gridDim.x) {
        const int64_t lt = item % ltiles, kc = item / ltiles;
        if (SIDE == 0) {
            // thread (tx, ty): line lt*32 + tx, inner indices kc*32 + ty + 8 u
            const int64_t line = lt * 32 + tx;
            const bool live = line < lines;
            const int E = live ? s.emax[line] : INT32_MIN;
            const bool dead = !live || E == INT32_MIN || s.nonfinite[line] < 0;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int64_t kk = kc * 32 + ty + 8 * u;
                uint32_t d = (!dead && kk < k) ? bound_digit(X[line + kk * ldx], E) : 0u;
                tile[tx][ty + 8 * u] = c_bound_code[d];
            }
            __syncthreads();
            // thread: line lt*32 + (threadIdx.x / 8), four bytes at kc*32 + 4 (threadIdx.x % 8)
            const int lr = threadIdx.x >> 3, kq = (threadIdx.x & 7) * 4;
            const int64_t oline = lt * 32 + lr, okk = kc * 32 + kq;
            if (oline < lines && okk < pitch)
                *reinterpret_cast<uint32_t *>(out + oline * pitch + okk) =
                    *reinterpret_cast<const uint32_t *>(&tile[lr][kq]);
            __syncthreads();
        } else {
            const int lr = threadIdx.x >> 3, kq = (threadIdx.x & 7) * 4;
            const int64_t line = lt * 32 + lr, kk0 = kc * 32 + kq;
            if (line >= lines || kk0 >= pitch) continue;
            const int E = s.emax[line];
            const bool dead = E == INT32_MIN || s.nonfinite[line] < 0;
            uint32_t word = 0u;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                uint32_t d = (!dead && kk0 + e < k) ? bound_digit(X[kk0 + e + line * ldx], E) : 0u;
                word |= static_cast<uint32_t>(c_bound_code[d]) << (8 * e);
            }
            *reinterpret_cast<uint32_t *>(out + line * pitch + kk0) = word;
        }
    }
}

// shift[line] of the accurate rule from the line's maximum of the bound product (the bit pattern of
// a non-negative integer-valued float, accumulated with atomicMax in the low word of sumsq[line]):
//   ((L - ceil(log2 max)) >> 1) + 4 - E
__global__ void accurate_finalize_kernel(ScanScratch s, int64_t lines, int L, int32_t *shift,
                                         unsigned int *status)
{
    int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x;
    if (i >= lines) return;
    if (s.nonfinite[i] < 0) {
        shift[i] = OZ_NONFINITE_SHIFT;
        atomicOr(status, 1u << OZ_ERR_NONFINITE_INPUT);
        return;
    }
    const int E = s.emax[i];
    if (E == INT32_MIN) { shift[i] = 0; return; }
    const uint32_t v = static_cast<uint32_t>(__uint_as_float(static_cast<uint32_t>(s.sumsq[i])));
    const int clog = v <= 1u ? 0 : 32 - __clz(static_cast<int>(v - 1u));
    shift[i] = ((L - clog) >> 1) + 4 - E;
}

// Four consecutive inner-dimension elements of one line -> 4 bytes of every stored plane.
template <int SET, int LAYOUT>
__device__ __forceinline__ void convert4(const double (&x)[4], int sigma, bool tz,
                                         const uint32_t *__restrict__ lut, uint8_t *out,
                                         int64_t plane_stride)
{
    uint32_t l0[4], l1[4], l2[4], l3[4];
    split_limbs4(x, sigma, tz, l0, l1, l2, l3);
    convert_all_moduli<SET, LAYOUT>(std::make_integer_sequence<int, set_r(SET)>{}, l0, l1, l2, l3, lut, out,
                            plane_stride);
}

template <int SET, int SIDE, int LAYOUT>
__global__ void __launch_bounds__(kConvThreads)
convert_kernel(const double *__restrict__ X, int64_t ldx, int64_t lines, int64_t k,
               const int32_t *__restrict__ shift, const uint32_t *__restrict__ lut_global,
               uint8_t *__restrict__ planes, int64_t plane_stride, int64_t row_pitch, int tz)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint32_t *lut = reinterpret_cast<uint32_t *>(smem_raw);
    for (int i = threadIdx.x; i < lut_words(SET); i += kConvThreads) lut[i] = lut_global[i];
    __syncthreads();

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // work items are numbered in 32 bits (checked on the host): cheap division
    const uint32_t nchunks = static_cast<uint32_t>((row_pitch + kChunk - 1) / kChunk);

    if (SIDE == 1) {
        const uint32_t items = static_cast<uint32_t>(lines) * nchunks;
        for (uint32_t item = blockIdx.x * 8u + warp; item < items; item += gridDim.x * 8u) {
            const uint32_t uline = item / nchunks;
            const int64_t line = uline;
            int64_t kb = static_cast<int64_t>(item - uline * nchunks) * kChunk + lane * 4;
            if (kb >= row_pitch) continue;
            int sigma = shift[line];
            bool dead = sigma == OZ_NONFINITE_SHIFT;
            double x[4];
#pragma unroll
            for (int e = 0; e < 4; ++e)
                x[e] = (!dead && kb + e < k) ? X[kb + e + line * ldx] : 0.0;
            convert4<SET, LAYOUT>(x, dead ? 0 : sigma, tz != 0, lut, planes + line * row_pitch + kb, plane_stride);
        }
    } else {
        double *tile = reinterpret_cast<double *>(smem_raw + lut_words(SET) * 4);
        const uint32_t ltiles = static_cast<uint32_t>((lines + kTileLines - 1) / kTileLines);
        const uint32_t items = ltiles * nchunks;
        for (uint32_t item = blockIdx.x; item < items; item += gridDim.x) {
            const uint32_t ukc = item / ltiles;
            const int64_t kc = ukc;
            const int64_t lt = item - ukc * ltiles;  // neighbouring blocks read neighbouring rows
            int64_t line_l = lt * kTileLines + lane;
            for (int kk = warp; kk < kChunk; kk += kConvThreads / 32) {
                int64_t kg = kc * kChunk + kk;
                tile[lane * kTilePitch + kk] =
                    (line_l < lines && kg < k) ? X[line_l + kg * ldx] : 0.0;
            }
            __syncthreads();
            int64_t kb = kc * kChunk + lane * 4;
#pragma unroll 1
            for (int li = warp * 4; li < warp * 4 + 4; ++li) {
                int64_t line = lt * kTileLines + li;
                if (line >= lines || kb >= row_pitch) continue;
                int sigma = shift[line];
                bool dead = sigma == OZ_NONFINITE_SHIFT;
                double x[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) x[e] = dead ? 0.0 : tile[li * kTilePitch + lane * 4 + e];
                convert4<SET, LAYOUT>(x, dead ? 0 : sigma, tz != 0, lut, planes + line * row_pitch + kb, plane_stride);
            }
            __syncthreads();
        }
    }
}

// ---- whole deconstruction of a group of lines in one kernel ------------------------------------
// When a few whole lines fit in shared memory next to the look-up table, a thread block loads them
// once and takes everything from there: largest exponent, the norm sums, the shift, and the
// conversion into planes.  The operand is then read from HBM once (8 bytes per element instead of
// 24 with the three-pass kernels above) and one launch replaces five.  The arithmetic is the same,
// function by function, so the outputs are identical; the sums are integers, hence independent of
// the order in which the warps add them.  Not for the accurate rule, whose shifts need the other
// operand.
struct FusedParams {
    const double *X;
    int64_t ldx, lines, k;
    int group;                 // lines per thread block pass
    int pitch;                 // doubles per line in shared memory (k + 1: conflict-free for both sides)
    int side, rule, tbits, tz;
    unsigned long long g2lo, g2hi;
    unsigned int esc_threshold;
    const uint32_t *lut_global;
    uint8_t *planes;
    int64_t plane_stride, row_pitch;
    int32_t *shift;
    unsigned int *status;
};

struct FusedLine {             // per-line results in shared memory
    unsigned long long sumsq;
    int emax, bad, shift;
    unsigned int l1;
};

template <int SET, int SIDE, int LAYOUT>
__global__ void __launch_bounds__(1024, 1)
deconstruct_fused_kernel(const __grid_constant__ FusedParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint32_t *lut = reinterpret_cast<uint32_t *>(smem_raw);
    double *buf = reinterpret_cast<double *>(smem_raw + lut_words(SET) * 4);
    FusedLine *res = reinterpret_cast<FusedLine *>(buf + static_cast<size_t>(p.group) * p.pitch);
    const int nthreads = blockDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = nthreads >> 5;
    for (int i = tid; i < lut_words(SET); i += nthreads) lut[i] = p.lut_global[i];
    const int64_t ngroups = (p.lines + p.group - 1) / p.group;
    const int k = static_cast<int>(p.k);
    for (int64_t g = blockIdx.x; g < ngroups; g += gridDim.x) {
        const int64_t line0 = g * p.group;
        const int nl = static_cast<int>(p.lines - line0 < p.group ? p.lines - line0 : p.group);
        __syncthreads();                 // the previous group's conversion has finished with buf / res
        // ---- load: nl lines x k doubles, coalesced along the operand's leading dimension
        if (SIDE == 0) {
            // element (line, kk) at X[line + kk ldx]: consecutive threads take consecutive lines
            // (the group size is a power of two on this side: shifts instead of divisions)
            const int gshift = 31 - __clz(p.group), gmask = p.group - 1;
            const int total = k << gshift;
            for (int e0 = tid; e0 < total; e0 += 4 * nthreads) {
                double v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int e = e0 + u * nthreads, kk = e >> gshift, l = e & gmask;
                    v[u] = (e < total && l < nl) ? p.X[line0 + l + static_cast<int64_t>(kk) * p.ldx] : 0.0;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int e = e0 + u * nthreads, kk = e >> gshift, l = e & gmask;
                    if (e < total && l < nl) buf[l * p.pitch + kk] = v[u];
                }
            }
        } else {
            // batches of independent loads: enough bytes in flight to run at memory speed
            for (int l0 = 0; l0 < nl; l0 += 4)
                for (int kk = tid; kk < k; kk += nthreads) {
                    double v[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) v[u] = l0 + u < nl ? p.X[kk + (line0 + l0 + u) * p.ldx] : 0.0;
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (l0 + u < nl) buf[(l0 + u) * p.pitch + kk] = v[u];
                }
        }
        if (tid < nl) {
            res[tid].sumsq = 0ull;
            res[tid].emax = INT32_MIN;
            res[tid].bad = 0;
            res[tid].l1 = 0u;
        }
        __syncthreads();
        // ---- the scans: a line is cut into `segs` pieces, one warp per piece
        const int segs = nwarps >= nl ? nwarps / nl : 1;
        const int span = (k + segs - 1) / segs;
        for (int item = warp; item < nl * segs; item += nwarps) {
            const int l = item / segs, seg = item - l * segs;
            const int k0 = seg * span, k1 = min(k, k0 + span);
            int emax = INT32_MIN, bad = 0;
            for (int kk = k0 + lane; kk < k1; kk += 32) {
                int e;
                const int c = classify(buf[l * p.pitch + kk], &e);
                if (c == 2) bad = 1;
                if (c == 1 && e > emax) emax = e;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                emax = max(emax, __shfl_xor_sync(0xFFFFFFFFu, emax, o));
                bad |= __shfl_xor_sync(0xFFFFFFFFu, bad, o);
            }
            if (lane == 0) {
                if (emax != INT32_MIN) atomicMax(&res[l].emax, emax);
                if (bad) atomicOr(&res[l].bad, 1);
            }
        }
        __syncthreads();
        if (p.rule == 1) {
            for (int item = warp; item < nl * segs; item += nwarps) {
                const int l = item / segs, seg = item - l * segs;
                const int k0 = seg * span, k1 = min(k, k0 + span);
                const int E = res[l].emax;
                if (E == INT32_MIN || res[l].bad) continue;              // warp-uniform
                const bool fast_scale = 9 - E >= -1000 && 9 - E <= 1000;
                const double scale9 = __hiloint2double((1023 + (fast_scale ? 9 - E : 0)) << 20, 0);
                unsigned long long acc = 0ull;
                unsigned int l1 = 0u;
                for (int kk = k0 + lane; kk < k1; kk += 32) {
                    const double x = buf[l * p.pitch + kk];
                    unsigned long long abar;
                    if (fast_scale) {
                        const double y = fabs(x) * scale9;
                        abar = static_cast<unsigned long long>(__double2ll_ru(y));
                        if (abar == 0ull && x != 0.0) abar = 1ull;
                    } else {
                        unsigned long long bits = static_cast<unsigned long long>(__double_as_longlong(x));
                        int be = static_cast<int>((bits >> 52) & 0x7FF);
                        unsigned long long frac = bits & 0xFFFFFFFFFFFFFull;
                        if (be == 0 && frac == 0) continue;
                        unsigned long long sig = be ? (frac | (1ull << 52)) : frac;
                        int ex = be ? be - 1023 : -1022;
                        int sh = 43 + E - ex;                 // |x| 2^(9-E) = sig / 2^sh
                        if (sh >= 64) abar = 1;
                        else if (sh <= 0) abar = sig << (-sh);
                        else abar = (sig >> sh) + ((sig & ((1ull << sh) - 1)) ? 1ull : 0ull);
                    }
                    acc += abar * abar;
                    l1 += static_cast<unsigned int>(abar);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
                    l1 += __shfl_xor_sync(0xFFFFFFFFu, l1, o);
                }
                if (lane == 0 && acc) {
                    atomicAdd(&res[l].sumsq, acc);
                    atomicAdd(&res[l].l1, l1);
                }
            }
            __syncthreads();
        }
        // ---- the shift of every line (same arithmetic as scan_finalize_kernel)
        if (tid < nl) {
            FusedLine &r = res[tid];
            int sh = 0;
            if (r.bad) {
                sh = OZ_NONFINITE_SHIFT;
                atomicOr(p.status, 1u << OZ_ERR_NONFINITE_INPUT);
            } else if (r.emax != INT32_MIN) {
                if (p.rule == 0) {
                    sh = p.tbits - 1 - r.emax;
                } else {
                    unsigned __int128 G2 = (static_cast<unsigned __int128>(p.g2hi) << 64) | p.g2lo;
                    unsigned __int128 q = G2 / static_cast<unsigned __int128>(r.sumsq);
                    unsigned long long qhi = static_cast<unsigned long long>(q >> 64);
                    unsigned long long qlo = static_cast<unsigned long long>(q);
                    int top = qhi ? 127 - __clzll(static_cast<long long>(qhi)) : 63 - __clzll(static_cast<long long>(qlo));
                    sh = (top >> 1) + 9 - r.emax;
                    const unsigned long long l1 = r.l1;
                    const unsigned __int128 flat = ((static_cast<unsigned __int128>(l1 * l1)) << 16) /
                                                   (static_cast<unsigned __int128>(static_cast<unsigned long long>(p.k)) * r.sumsq);
                    atomicMin(p.status + 1 + p.side, static_cast<unsigned int>(flat));
                    p.status[3] = p.esc_threshold;
                }
            }
            r.shift = sh;
            p.shift[line0 + tid] = sh;
        }
        __syncthreads();
        // ---- conversion: a thread takes four consecutive inner indices of one line
        const int quads = static_cast<int>(p.row_pitch >> 2);          // row_pitch is a multiple of 16
        for (int it = tid; it < nl * quads; it += nthreads) {
            const int l = it / quads, kb = (it - l * quads) * 4;
            const int sigma = res[l].shift;
            const bool dead = sigma == OZ_NONFINITE_SHIFT;
            double x[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) x[e] = (!dead && kb + e < k) ? buf[l * p.pitch + kb + e] : 0.0;
            convert4<SET, LAYOUT>(x, dead ? 0 : sigma, p.tz != 0, lut, p.planes + (line0 + l) * p.row_pitch + kb,
                                  p.plane_stride);
        }
    }
}

// Lines per thread-block pass of the fused kernel and its launch shape; group = 0: not applicable
// (the lines are too long for shared memory).
#ifndef OZ_FUSED_MAX_ELEMS
#define OZ_FUSED_MAX_ELEMS (1ll << 22)
#endif
struct FusedShape { int group, threads, grid; size_t smem; };

FusedShape fused_shape(int set, int side, int64_t lines, int64_t k, int sms)
{
    FusedShape f{0, 0, 0, 0};
    if (k < 1 || k > 32768 || lines < 1) return f;
    // The one-kernel form wins where the call is bound by launch latency; larger operands keep the
    // three-pass kernels, whose many small blocks hide the memory latency better.
    if (lines * k > OZ_FUSED_MAX_ELEMS) return f;
    const size_t line_bytes = static_cast<size_t>(k + 1) * 8;
    const size_t fixed = lut_words(set) * 4 + 64 * sizeof(FusedLine) + 64;
    // two blocks per SM when lines are short enough for that, else one block with more threads
    const size_t budget2 = 110 * 1024, budget1 = 224 * 1024;
    int group = static_cast<int>((budget2 - fixed) / line_bytes);
    int threads = 512;
    const int min_group = side == 0 ? 4 : 1;         // side 0 loads `group` consecutive doubles per inner index
    if (group < (side == 0 ? 8 : 2)) {
        group = static_cast<int>((budget1 - fixed) / line_bytes);
        threads = 1024;
    }
    if (group < min_group) return f;
    if (group > 32) group = 32;
    // small operands: fewer lines per block, so that the blocks cover the machine (a 256 x 256 operand
    // with 32 lines per block would run on 8 SMs)
#ifndef OZ_FUSED_SPREAD_MIN
#define OZ_FUSED_SPREAD_MIN 8
#endif
    {
        const int64_t blocks_wanted = static_cast<int64_t>(sms) * (threads == 512 ? 2 : 1);
        int64_t spread = (lines + blocks_wanted - 1) / blocks_wanted;
        const int floor_group = side == 0 ? OZ_FUSED_SPREAD_MIN : 1;
        if (spread < floor_group) spread = floor_group;
        if (spread < group) group = static_cast<int>(spread);
    }
    if (side == 0) {
        int pow2 = 1;
        while (pow2 * 2 <= group) pow2 *= 2;
        group = pow2;
    } else if (group > lines) {
        group = static_cast<int>(lines);
    }
    f.group = group;
    f.threads = threads;
    f.smem = fixed + static_cast<size_t>(group) * line_bytes;
    const int64_t ngroups = (lines + group - 1) / group;
    const int64_t cap = static_cast<int64_t>(sms) * (threads == 512 ? 2 : 1);
    f.grid = static_cast<int>(ngroups < cap ? ngroups : cap);
    return f;
}

template <int SET, int SIDE, int LAYOUT>
oz_status_t launch_fused(const FusedParams &p, const FusedShape &f, cudaStream_t stream)
{
    auto kernel = deconstruct_fused_kernel<SET, SIDE, LAYOUT>;
    OZ_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(f.smem)));
    kernel<<<f.grid, f.threads, f.smem, stream>>>(p);
    count_launch();
    OZ_CUDA_CHECK(cudaGetLastError());
    return OZ_OK;
}

template <int SET, int SIDE, int LAYOUT>
oz_status_t launch_convert(const double *X, int64_t ldx, int64_t lines, int64_t k,
                           const int32_t *shift, const uint32_t *lut, uint8_t *planes,
                           int64_t plane_stride, int64_t row_pitch, int tz, cudaStream_t stream)
{
    size_t smem = lut_words(SET) * 4 + (SIDE == 0 ? sizeof(double) * kTileLines * kTilePitch : 0);
    OZ_CUDA_CHECK(cudaFuncSetAttribute(convert_kernel<SET, SIDE, LAYOUT>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(smem)));
    int64_t nchunks = (row_pitch + kChunk - 1) / kChunk;
    if (lines * nchunks >= 0x7FFFFFFFll) return OZ_ERR_UNSUPPORTED;   // item numbers are 32-bit
    int64_t need = SIDE == 1 ? (lines * nchunks + 7) / 8
                             : ((lines + kTileLines - 1) / kTileLines) * nchunks;
    int dev = 0, sms = 148;
    OZ_CUDA_CHECK(cudaGetDevice(&dev));
    OZ_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    // persistent blocks: as many as are resident at once (each copies the table once)
    int per_sm = 1;
    OZ_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, convert_kernel<SET, SIDE, LAYOUT>,
                                                                kConvThreads, smem));
    int64_t cap = static_cast<int64_t>(sms) * (per_sm > 0 ? per_sm : 1);
    int grid = static_cast<int>(need < cap ? need : cap);
    convert_kernel<SET, SIDE, LAYOUT><<<grid, kConvThreads, smem, stream>>>(
        X, ldx, lines, k, shift, lut, planes, plane_stride, row_pitch, tz);
    count_launch();
    OZ_CUDA_CHECK(cudaGetLastError());
    return OZ_OK;
}

}  // namespace

// scan_init + the scan passes of the route's scale rule [+ the shifts, except for the accurate rule,
// whose shifts come later from the bound product]
oz_status_t launch_scan(int side, int64_t lines, int64_t k, const double *X, int64_t ldx, int set,
                        const Route &rt, int32_t *shift, void *scratch, cudaStream_t stream)
{
    ScanScratch s = carve_scratch(scratch, lines);
    unsigned int *status = device_status_word();
    int blocks1d = static_cast<int>((lines + 255) / 256);
    scan_init_kernel<<<blocks1d, 256, 0, stream>>>(s, lines);
    count_launch();

    // split the inner dimension so that the scan fills the machine even for few lines
    int64_t line_blocks = side == 0 ? (lines + 255) / 256 : (lines + 7) / 8;
    int64_t want_split = (148 * 8 + line_blocks - 1) / line_blocks;
    int64_t max_split = (k + 63) / 64;
    int64_t split = want_split < max_split ? want_split : max_split;
    if (split < 1) split = 1;
    if (split > 65535) split = 65535;
    int64_t kspan = (k + split - 1) / split;
    split = k > 0 ? (k + kspan - 1) / kspan : 0;

    int tA = 0, tB = 0;
    budget_maxexp(set, k, &tA, &tB);
    uint64_t g2lo = 0, g2hi = 0;
    cs_bound_squared(set, k, &g2lo, &g2hi);

    if (k > 0) {
        dim3 grid(static_cast<unsigned>(line_blocks), static_cast<unsigned>(split));
        if (side == 0) scan_kernel<0, 0><<<grid, 256, 0, stream>>>(X, ldx, lines, k, kspan, s);
        else scan_kernel<1, 0><<<grid, 256, 0, stream>>>(X, ldx, lines, k, kspan, s);
        count_launch();
        if (rt.rule == 1) {
            if (side == 0) scan_kernel<0, 1><<<grid, 256, 0, stream>>>(X, ldx, lines, k, kspan, s);
            else scan_kernel<1, 1><<<grid, 256, 0, stream>>>(X, ldx, lines, k, kspan, s);
            count_launch();
        }
    }
    if (rt.rule != 2) {
        scan_finalize_kernel<<<blocks1d, 256, 0, stream>>>(s, lines, k, side, rt.rule, side == 0 ? tA : tB, g2lo,
                                                           g2hi, esc_threshold(set), shift, status);
        count_launch();
    }
    OZ_CUDA_CHECK(cudaGetLastError());
    return OZ_OK;
}

// accurate rule: the line's magnitude digits as one K-major E4M3 plane (after launch_scan)
oz_status_t launch_bound_plane(int side, int64_t lines, int64_t k, const double *X, int64_t ldx,
                               void *scratch, uint8_t *plane, int64_t pitch, cudaStream_t stream)
{
    ScanScratch s = carve_scratch(scratch, lines);
    int dev = 0, sms = 148;
    OZ_CUDA_CHECK(cudaGetDevice(&dev));
    OZ_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const int64_t need = ((lines + 31) / 32) * ((pitch + 31) / 32);
    const int64_t cap = static_cast<int64_t>(sms) * 8;
    const int grid = static_cast<int>(need < cap ? need : cap);
    if (side == 0) bound_plane_kernel<0><<<grid, 256, 0, stream>>>(X, ldx, lines, k, s, plane, pitch);
    else bound_plane_kernel<1><<<grid, 256, 0, stream>>>(X, ldx, lines, k, s, plane, pitch);
    count_launch();
    OZ_CUDA_CHECK(cudaGetLastError());
    return OZ_OK;
}

// accurate rule: where the bound product accumulates the maximum of line `l` (a 32-bit word, zero
// after launch_scan): word stride 2 from this address
unsigned int *bound_maxima(void *scratch, int64_t lines)
{
    return reinterpret_cast<unsigned int *>(carve_scratch(scratch, lines).sumsq);
}

// accurate rule: shifts from the maxima of the bound product
oz_status_t launch_accurate_finalize(int64_t lines, void *scratch, int budget_log2, int32_t *shift,
                                     cudaStream_t stream)
{
    ScanScratch s = carve_scratch(scratch, lines);
    accurate_finalize_kernel<<<static_cast<int>((lines + 255) / 256), 256, 0, stream>>>(s, lines, budget_log2, shift,
                                                                                         device_status_word());
    count_launch();
    OZ_CUDA_CHECK(cudaGetLastError());
    return OZ_OK;
}

oz_status_t upload_bound_codes(const unsigned char *codes33)
{
    OZ_CUDA_CHECK(cudaMemcpyToSymbol(c_bound_code, codes33, 33));
    return OZ_OK;
}

// quantise, reduce, look up, store: the planes of one operand from its shifts
oz_status_t launch_convert_planes(int side, int64_t lines, int64_t k, const double *X, int64_t ldx,
                                  int set, const Route &rt, uint8_t *planes, int64_t plane_stride,
                                  int64_t row_pitch, const int32_t *shift, cudaStream_t stream)
{
    const uint32_t *lut = device_lut(set, rt.substrate);
#define OZ_CONVERT(SET_, SIDE_, LAYOUT_)                                                                 \
    launch_convert<SET_, SIDE_, LAYOUT_>(X, ldx, lines, k, shift, lut, planes, plane_stride, row_pitch, \
                                         rt.quant, stream)
#define OZ_CONVERT_SET(SET_)                                                                             \
    (side == 1 ? (layout == kLayoutMergedI8B ? OZ_CONVERT(SET_, 1, kLayoutMergedI8B)                    \
                                             : OZ_CONVERT(SET_, 1, kLayoutDigits))                      \
               : (layout == kLayoutMerged      ? OZ_CONVERT(SET_, 0, kLayoutMerged)                     \
                  : layout == kLayoutMergedI8A ? OZ_CONVERT(SET_, 0, kLayoutMergedI8A)                  \
                                               : OZ_CONVERT(SET_, 0, kLayoutDigits)))
    const int layout = rt.layout(side);
    if (layout == kLayoutNative) return side == 0 ? OZ_CONVERT(2, 0, kLayoutNative) : OZ_CONVERT(2, 1, kLayoutNative);
    if (set == 0) return OZ_CONVERT_SET(0);
    if (set == 1) return OZ_CONVERT_SET(1);
    return OZ_CONVERT_SET(2);
#undef OZ_CONVERT_SET
#undef OZ_CONVERT
}

oz_status_t launch_deconstruct(int side, int64_t lines, int64_t k, const double *X, int64_t ldx,
                               int set, const Route &rt, uint8_t *planes, int64_t plane_stride,
                               int64_t row_pitch, int32_t *shift, void *scratch,
                               cudaStream_t stream)
{
    if (rt.rule == 2) return OZ_ERR_UNSUPPORTED;      // the accurate rule needs both operands
    int dev = 0, sms = 148;
    OZ_CUDA_CHECK(cudaGetDevice(&dev));
    OZ_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const FusedShape f = fused_shape(rt.layout(side) == kLayoutNative ? 2 : set, side, lines, k, sms);
    if (f.group > 0 && !rt.fallback) {      // the row check reads the scan results of the three-pass form
        FusedParams p{};
        p.X = X; p.ldx = ldx; p.lines = lines; p.k = k;
        p.group = f.group;
        p.pitch = static_cast<int>(k + 1);
        p.side = side; p.rule = rt.rule; p.tz = rt.quant;
        int tA = 0, tB = 0;
        budget_maxexp(set, k, &tA, &tB);
        p.tbits = side == 0 ? tA : tB;
        uint64_t g2lo = 0, g2hi = 0;
        cs_bound_squared(set, k, &g2lo, &g2hi);
        p.g2lo = g2lo; p.g2hi = g2hi;
        p.esc_threshold = esc_threshold(set);
        p.lut_global = device_lut(set, rt.substrate);
        p.planes = planes; p.plane_stride = plane_stride; p.row_pitch = row_pitch;
        p.shift = shift;
        p.status = device_status_word();
        const int layout = rt.layout(side);
#define OZ_FUSED(SET_, SIDE_, LAYOUT_) launch_fused<SET_, SIDE_, LAYOUT_>(p, f, stream)
#define OZ_FUSED_SET(SET_)                                                                      \
    (side == 1 ? (layout == kLayoutMergedI8B ? OZ_FUSED(SET_, 1, kLayoutMergedI8B)             \
                                             : OZ_FUSED(SET_, 1, kLayoutDigits))               \
               : (layout == kLayoutMerged      ? OZ_FUSED(SET_, 0, kLayoutMerged)              \
                  : layout == kLayoutMergedI8A ? OZ_FUSED(SET_, 0, kLayoutMergedI8A)           \
                                               : OZ_FUSED(SET_, 0, kLayoutDigits)))
        if (layout == kLayoutNative) return side == 0 ? OZ_FUSED(2, 0, kLayoutNative) : OZ_FUSED(2, 1, kLayoutNative);
        if (set == 0) return OZ_FUSED_SET(0);
        if (set == 1) return OZ_FUSED_SET(1);
        return OZ_FUSED_SET(2);
#undef OZ_FUSED_SET
#undef OZ_FUSED
    }
    oz_status_t st = launch_scan(side, lines, k, X, ldx, set, rt, shift, scratch, stream);
    if (st != OZ_OK) return st;
    return launch_convert_planes(side, lines, k, X, ldx, set, rt, planes, plane_stride, row_pitch, shift, stream);
}

// flags, ordered list and number of the rows that go to the native FP64 path, from the scan results
// that the three-pass deconstruction of both operands left in their scratch blocks
oz_status_t launch_esc_rows(void *scratchA, int64_t m, void *scratchB, int64_t n, int64_t k, int set,
                            unsigned char *flag, int *list, unsigned int *count, cudaStream_t stream)
{
    esc_rows_kernel<<<1, 1024, 0, stream>>>(carve_scratch(scratchA, m), m, carve_scratch(scratchB, n), n, k,
                                            esc_threshold(set), flag, list, count, device_status_word());
    count_launch();
    OZ_CUDA_CHECK(cudaGetLastError());
    return OZ_OK;
}

}  // namespace oz
