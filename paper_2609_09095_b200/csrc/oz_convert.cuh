// Conversion of quantised FP64 elements into plane bytes (Algorithm 2: residues of every modulus from
// the 16-bit limbs of the integer, digit split and plane codes by table look-up), shared by the
// deconstruction kernels and by the product kernel that converts its A operand on the fly.
// Internal to liboz_b200.so; every function is device-inline and lives in the including file's
// anonymous namespace.
#pragma once

#include <utility>

#include "oz_internal.h"

namespace oz {
namespace {

// Eq. 1 for one element, fast form: multiplying by the power of two 2^sigma is exact in FP64 (a
// product that underflows is far below 1/2 and rounds to zero either way), and the hardware
// conversion rounds to nearest-even or toward zero.  Valid while 2^sigma is a normal double.
__device__ __forceinline__ long long quantise_fp(double x, double scale, bool tz)
{
    double y = x * scale;
    return tz ? __double2ll_rz(y) : __double2ll_rn(y);
}

// Eq. 1 for one element, integer form (any sigma): a' = quant(x 2^sigma) as a 64-bit integer.
__device__ __forceinline__ long long quantise(double x, int sigma, bool tz)
{
    unsigned long long bits = static_cast<unsigned long long>(__double_as_longlong(x));
    int be = static_cast<int>((bits >> 52) & 0x7FF);
    unsigned long long frac = bits & 0xFFFFFFFFFFFFFull;
    unsigned long long sig = be ? (frac | (1ull << 52)) : frac;
    int ex = be ? be - 1023 : -1022;
    int sh = 52 - ex - sigma;                       // |x| 2^sigma = sig / 2^sh
    unsigned long long q;
    if (sh <= 0) {
        q = sig << (sh < -63 ? 63 : -sh);
    } else {
        if (sh > 63) sh = 63;                       // sig < 2^53: anything past 54 rounds to zero
        if (tz) q = sig >> sh;
        else q = (sig + ((1ull << (sh - 1)) - 1ull) + ((sig >> sh) & 1ull)) >> sh;  // ties to even
    }
    return (bits >> 63) ? -static_cast<long long>(q) : static_cast<long long>(q);
}

// One modulus (compile-time index I of set SET) for four consecutive inner-dimension elements:
// residues, table look-up, byte transposition, 2 or 3 four-byte plane stores.
template <int SET, int LAYOUT, int I>
__device__ __forceinline__ void convert_modulus(const uint32_t (&l0)[4], const uint32_t (&l1)[4],
                                                const uint32_t (&l2)[4], const uint32_t (&l3)[4],
                                                const uint32_t *__restrict__ lut, uint8_t *out,
                                                int64_t plane_stride)
{
    constexpr uint32_t m = modulus(SET, I);
    constexpr uint32_t c1 = pow2_mod(16, m), c2 = pow2_mod(32, m), c3 = pow2_mod(48, m);
    // a' = l0 + l1 2^16 + l2 2^32 + l3 2^48 with the top limb SIGNED; `bias` (a multiple of m not
    // below 2^15 c3) keeps the limb sum non-negative, so no separate sign correction is needed.
    constexpr uint32_t bias = ((32768u * c3 + m - 1) / m) * m;
    static_assert(65535ull * (1ull + c1 + c2) + 32767ull * c3 + bias < (1ull << 28), "limb sum below 2^28");
    // Everything is carried four times too large, so that the remainder is the BYTE offset of the
    // table entry: v = 4 (limb sum) < 2^30, and floor(v / 4m) = (v * ceil(2^(32+s) / 4m)) >> (32+s)
    // exactly for s = ceil(log2 m) (the multiplier stays below 2^31).
    // Per element: four multiply-adds, one multiply-high, a shift, one multiply-subtract, one look-up.
    constexpr uint32_t m4 = 4u * m;
    constexpr int s = ceil_log2(m);
    constexpr uint32_t magic = static_cast<uint32_t>(((1ull << (32 + s)) + m4 - 1) / m4);
    static_assert(static_cast<unsigned long long>(m4) << 30 <= (1ull << (32 + s)), "exact quotient for v < 2^30");
    constexpr int off = lut_offset(SET, I);
    constexpr int plane = first_plane(SET, I, LAYOUT);
    const unsigned char *table = reinterpret_cast<const unsigned char *>(lut + off);
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        uint32_t v = l3[e] * (4u * c3) + 4u * bias;      // l3 holds the signed limb in two's complement
        v = l2[e] * (4u * c2) + v;
        v = l1[e] * (4u * c1) + v;
        v = l0[e] * 4u + v;
        const uint32_t r4 = v - (__umulhi(v, magic) >> s) * m4;        // 4 (a' mod m), canonical
        w[e] = *reinterpret_cast<const uint32_t *>(table + r4);
    }
    uint32_t t01 = __byte_perm(w[0], w[1], 0x5140);
    uint32_t t23 = __byte_perm(w[2], w[3], 0x5140);
    const uint32_t first = __byte_perm(t01, t23, 0x5410), second = __byte_perm(t01, t23, 0x7632);
    if (LAYOUT == kLayoutNative) {            // one plane: the centred residue itself
        *reinterpret_cast<uint32_t *>(out + plane * plane_stride) = first;
        return;
    }
    if (planes_of(m) == 3) {
        // bytes 2 and 3 of the table words: d0+d1 and the byte the merged layouts swap in
        // (FP8: the pre-scaled -16*d1 for d1; INT8: -d0 for d0, with 4*d1 made by a byte-wise shift)
        uint32_t u01 = __byte_perm(w[0], w[1], 0x7362);
        uint32_t u23 = __byte_perm(w[2], w[3], 0x7362);
        const uint32_t extra = __byte_perm(u01, u23, 0x7632);
        constexpr bool kI8 = LAYOUT == kLayoutMergedI8A || LAYOUT == kLayoutMergedI8B;
        *reinterpret_cast<uint32_t *>(out + plane * plane_stride) = LAYOUT == kLayoutMergedI8A ? extra : first;
        *reinterpret_cast<uint32_t *>(out + (plane + 1) * plane_stride) =
            LAYOUT == kLayoutMerged ? extra : (kI8 ? ((second << 2) & 0xFCFCFCFCu) : second);
        *reinterpret_cast<uint32_t *>(out + (plane + 2) * plane_stride) = __byte_perm(u01, u23, 0x5410);
    } else {
        *reinterpret_cast<uint32_t *>(out + plane * plane_stride) = first;
        *reinterpret_cast<uint32_t *>(out + (plane + 1) * plane_stride) = second;
    }
}

template <int SET, int LAYOUT, int... I>
__device__ __forceinline__ void convert_all_moduli(std::integer_sequence<int, I...>,
                                                   const uint32_t (&l0)[4], const uint32_t (&l1)[4],
                                                   const uint32_t (&l2)[4], const uint32_t (&l3)[4],
                                                   const uint32_t *__restrict__ lut, uint8_t *out,
                                                   int64_t plane_stride)
{
    (convert_modulus<SET, LAYOUT, I>(l0, l1, l2, l3, lut, out, plane_stride), ...);
}

// The four 16-bit limbs (top one signed) of the quantised values of four elements.
__device__ __forceinline__ void split_limbs4(const double (&x)[4], int sigma, bool tz, uint32_t (&l0)[4],
                                             uint32_t (&l1)[4], uint32_t (&l2)[4], uint32_t (&l3)[4])
{
    // 2^sigma as a double when it is a normal number (always, except for lines of subnormals)
    const bool fast = sigma >= -1000 && sigma <= 1000;
    const double scale = __hiloint2double((1023 + (fast ? sigma : 0)) << 20, 0);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        long long a = fast ? quantise_fp(x[e], scale, tz) : quantise(x[e], sigma, tz);
        unsigned long long p = static_cast<unsigned long long>(a);
        uint32_t lo = static_cast<uint32_t>(p), hi = static_cast<uint32_t>(p >> 32);
        l0[e] = lo & 0xFFFFu;
        l1[e] = lo >> 16;
        l2[e] = hi & 0xFFFFu;
        l3[e] = static_cast<uint32_t>(static_cast<int32_t>(hi) >> 16);   // signed top limb
    }
}

}  // namespace
}  // namespace oz
