// Reconstruction with the CRT recombination hosted on the INT8 tensor pipe (Algorithm 3, the
// "[INT8-TENSOR + SIMT] mixed-radix reconstruction ... ~r MACs/output as a length-r recombination on
// the INT8 tensor pipe plus a few SIMT carry/normalise ops; single rounding to FP64").
//
// CRT fixes c' uniquely, so, as in the FP64 kernel, the weighted form is evaluated:
//     S = sum_i c_i V_i,   V_i = ((M/m_i)^-1 mod m_i) (M/m_i),   c' = S - kappa M  lifted to [-M/2, M/2).
// Here S is formed in integers.  With c_i cut into bytes c_{i,a} and V_i into bytes V_{i,b},
//     S = sum_s 2^(8 s) P_s,      P_s = sum_{i, a, b : a + b = s} c_{i,a} V_{i,b},
// and the sixteen P_s of one output are one row of a small matrix product
//     P[output][s] = sum_K A[output][K] B[s][K],   K = (i, a),  A = residue bytes,  B[s][(i,a)] = V_{i, s-a},
// an unsigned 8-bit product with K = 32 that the tensor core takes in ONE instruction per 128 outputs
// (tcgen05.mma kind::i8, M = 128, N = 16, K = 32, operands in shared memory, accumulator in TMEM).
// Every P_s is below 2^21, exact in INT32.  TMEM lane l holds the sixteen sums of the output that
// thread l packed, so each thread reads its own row back (tcgen05.ld) and finishes alone:
// carry-propagate the P_s into a 160-bit integer, subtract kappa M (kappa from the leading bits,
// corrected by comparison), lift, and round once to FP64 in integer arithmetic (nearest, ties to
// even, through the 64 leading bits and a sticky bit).  No FP64 arithmetic except the update of C.
//
// The residues come in the tile-ordered private layout of the whole-method calls (ResidueTiling): a
// thread block of 128 threads takes 128 consecutive words of a 32 x 64 patch, i.e. ROWS = 2 (uint16
// residues) or 4 (uint8) outputs per thread, ROWS small products per step.
//
// Every wait is bounded; on expiry the block records OZ_ERR_TIMEOUT, frees its TMEM and returns.
#include "oz_internal.h"

namespace oz {
namespace {

struct HostedConst {
    unsigned char B[16][32];   // B[s][K]
    uint32_t M[4];             // M, 32-bit limbs, least significant first (M < 2^118)
    uint32_t Mh[4];            // M / 2
    float kappa_scale;         // 2^top_shift / M, rounded down
    int top_shift;             // S >> top_shift is below 2^30
};

__constant__ HostedConst c_hosted[kNumSets];

__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// shared-memory matrix descriptor, K-major, no swizzle: 8-row x 16-byte core matrices of 128
// contiguous bytes; the next core matrix along K is `lbo` bytes on, the next 8-row group `sbo` bytes
__device__ __forceinline__ uint64_t plain_desc(uint32_t addr, uint32_t lbo, uint32_t sbo)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((addr >> 4) & 0x3FFFu);
    d |= static_cast<uint64_t>((lbo >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>((sbo >> 4) & 0x3FFFu) << 32;
    d |= static_cast<uint64_t>(1) << 46;                 // descriptor version of sm_100
    return d;                                            // bits 61..63 = 0: no swizzle
}

// instruction descriptor: D = s32, A = B = u8, both K-major, N = 16, M = 128
constexpr uint32_t kHostedIdesc = (2u << 4) | (0u << 7) | (0u << 10) | (static_cast<uint32_t>(16 >> 3) << 17) |
                                  (static_cast<uint32_t>(128 >> 4) << 24);

__device__ __forceinline__ void mma_u8(uint32_t d_tmem, uint64_t da, uint64_t db)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 0, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(da), "l"(db), "r"(kHostedIdesc) : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
          "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
          "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ bool bar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

__device__ __forceinline__ unsigned long long timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// x * 2^scale for a finite double x (exact unless the result leaves the normal range)
__device__ __forceinline__ double scale_by_pow2(double x, int scale)
{
    int hi = __double2hiint(x);
    int be = (hi >> 20) & 0x7FF;
    int nb = be + scale;
    if (be != 0 && nb >= 1 && nb <= 2046) return __hiloint2double(hi + (scale << 20), __double2loint(x));
    return scalbn(x, scale);
}

// The sixteen byte-position sums of one output -> its FP64 value P = RN(c' 2^-shift_sum).
template <int SET>
__device__ __forceinline__ double finish_from_sums(const uint32_t (&P)[16], int shift_sum)
{
    const HostedConst &K = c_hosted[SET];
    // S = sum_s P_s 2^(8 s): four 64-bit partial sums of weight 2^0, 2^32, 2^64, 2^96 (each < 2^47)
    unsigned long long acc[4];
#pragma unroll
    for (int g = 0; g < 4; ++g)
        acc[g] = static_cast<unsigned long long>(P[4 * g]) + (static_cast<unsigned long long>(P[4 * g + 1]) << 8) +
                 (static_cast<unsigned long long>(P[4 * g + 2]) << 16) + (static_cast<unsigned long long>(P[4 * g + 3]) << 24);
    uint32_t L[5];
    unsigned long long t = acc[0];
    L[0] = static_cast<uint32_t>(t);
    t = (t >> 32) + acc[1];
    L[1] = static_cast<uint32_t>(t);
    t = (t >> 32) + acc[2];
    L[2] = static_cast<uint32_t>(t);
    t = (t >> 32) + acc[3];
    L[3] = static_cast<uint32_t>(t);
    L[4] = static_cast<uint32_t>(t >> 32);
    // kappa = floor(S / M) or one less, from the 30 leading bits (every rounding is downwards)
    const unsigned long long top64 = (static_cast<unsigned long long>(L[4]) << 32) | L[3];
    const uint32_t top = static_cast<uint32_t>(top64 >> (K.top_shift - 96));
    const uint32_t kappa = __float2uint_rz(__fmul_rz(__uint2float_rz(top), K.kappa_scale));
    // R = S - kappa M  (non-negative, below 2 M)
    uint32_t R[5];
    unsigned long long mulc = 0;
    long long carry = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const unsigned long long prod = static_cast<unsigned long long>(kappa) * K.M[i] + mulc;
        mulc = prod >> 32;
        const long long d = static_cast<long long>(L[i]) - static_cast<long long>(static_cast<uint32_t>(prod)) + carry;
        R[i] = static_cast<uint32_t>(d);
        carry = d >> 32;
    }
    R[4] = static_cast<uint32_t>(static_cast<long long>(L[4]) - static_cast<long long>(mulc) + carry);
    // at most one more M to take off (two iterations allowed for safety)
#pragma unroll 1
    for (int it = 0; it < 2; ++it) {
        bool ge = R[4] != 0u;
        if (!ge) {
            ge = true;                       // R >= M ?  compare from the top limb down
#pragma unroll
            for (int i = 3; i >= 0; --i) {
                if (R[i] != K.M[i]) { ge = R[i] > K.M[i]; break; }
            }
        }
        if (!ge) break;
        long long b = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const long long d = static_cast<long long>(R[i]) - static_cast<long long>(K.M[i]) + b;
            R[i] = static_cast<uint32_t>(d);
            b = d >> 32;
        }
        R[4] = static_cast<uint32_t>(static_cast<long long>(R[4]) + b);
    }
    // lift to [-M/2, M/2): c' = R - M when R >= M/2
    bool neg = true;
#pragma unroll
    for (int i = 3; i >= 0; --i) {
        if (R[i] != K.Mh[i]) { neg = R[i] > K.Mh[i]; break; }
    }
    if (neg) {
        long long b = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const long long d = static_cast<long long>(K.M[i]) - static_cast<long long>(R[i]) + b;
            R[i] = static_cast<uint32_t>(d);
            b = d >> 32;
        }
    }
    // |c'| -> nearest double, ties to even: the 64 leading bits with a sticky bit, converted once
    const unsigned long long hi = (static_cast<unsigned long long>(R[3]) << 32) | R[2];
    const unsigned long long lo = (static_cast<unsigned long long>(R[1]) << 32) | R[0];
    double d;
    int scale;
    if (hi == 0ull) {
        if (lo == 0ull) return 0.0;
        d = __ull2double_rn(lo);
        scale = 0;
    } else {
        const int lz = __clzll(static_cast<long long>(hi));
        const unsigned long long lead = lz ? ((hi << lz) | (lo >> (64 - lz))) : hi;
        const unsigned long long rest = lo << lz;
        d = __ull2double_rn(lead | (rest ? 1ull : 0ull));
        scale = 64 - lz;
    }
    d = scale_by_pow2(d, scale - shift_sum);
    return neg ? -d : d;
}

template <int SET>
__global__ void __launch_bounds__(128)
reconstruct_hosted_kernel(const void *__restrict__ Rv, int cg, int tiles_n, int tn0, int ntn, int tiles_m,
                          int64_t m, int64_t n, int64_t col0, int64_t col1,
                          const int32_t *__restrict__ shiftA, const int32_t *__restrict__ shiftB,
                          double alpha, double beta, double *__restrict__ C, int64_t ldc, int vecC,
                          unsigned int *status)
{
    constexpr int RB = residue_bytes(SET), ROWS = 4 / RB, r = set_r(SET);
    constexpr int kBlockWords = 64 * 32 * RB / 4;          // words of one 32 x 64 patch per modulus
    constexpr int kPieces = kBlockWords / 128;             // 128-word pieces of a patch: 8 or 4
    constexpr uint32_t kTmemCols = ROWS * 16 < 32 ? 32 : ROWS * 16;
    __shared__ __align__(128) unsigned char tileA[ROWS][128 * 32];
    __shared__ __align__(128) unsigned char tileB[16 * 32];
    __shared__ __align__(8) unsigned long long bar_storage;
    __shared__ uint32_t tmem_slot;
    const int t = threadIdx.x, warp = t >> 5;
    const uint32_t bar = smem_addr(&bar_storage);

    // B: byte (s, K) of the constant matrix into its core-matrix position
    for (int e = t; e < 16 * 32; e += 128) {
        const int s = e >> 5, kb = e & 31;
        tileB[(s >> 3) * 256 + (kb >> 4) * 128 + (s & 7) * 16 + (kb & 15)] = c_hosted[SET].B[s][kb];
    }
    if (t == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(1));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_slot;
    const uint64_t descB = plain_desc(smem_addr(tileB), 128, 256);

    const int64_t total = static_cast<int64_t>(tiles_m) * ntn * cg * 16 * kPieces;
    uint32_t phase = 0;
    bool alive = true;
    for (int64_t work = blockIdx.x; alive && work < total; work += gridDim.x) {
        // block-uniform decode of the piece
        uint32_t u = static_cast<uint32_t>(work % (static_cast<int64_t>(kPieces) * 16 * cg));
        const int64_t tile = work / (static_cast<int64_t>(kPieces) * 16 * cg);
        const uint32_t piece = u % kPieces; u /= kPieces;
        const uint32_t wi = u & 15u, rank = u >> 4;
        const uint32_t tn = static_cast<uint32_t>(tn0) + static_cast<uint32_t>(tile % ntn);
        const uint32_t tm = static_cast<uint32_t>(tile / ntn);
        const uint32_t w_idx = piece * 128u + t;
        const uint32_t lane = (w_idx >> 2) & 31u, sub = w_idx & 3u;
        const int64_t row = static_cast<int64_t>(tm) * 256 + (wi >> 2) * 64 + piece * (16 / RB) + sub * ROWS;
        const int64_t j = (static_cast<int64_t>(tn) * cg + rank) * 128 + (wi & 3u) * 32 + lane;
        const bool valid = row < m && j < n && j >= col0 && j < col1;
        const int64_t wb = ((static_cast<int64_t>(tm) * tiles_n + tn) * cg + rank) * 16 + wi;
        const unsigned char *base = static_cast<const unsigned char *>(Rv) + ((wb * r) * kBlockWords + w_idx) * 4;
        uint32_t w[16];
#pragma unroll
        for (int i = 0; i < 16; ++i)
            w[i] = (i < r && valid) ? *reinterpret_cast<const uint32_t *>(base + i * (kBlockWords * 4)) : 0u;
        // old values of C and the shifts travel while the tensor core works
        const int nrows = valid ? (m - row < ROWS ? static_cast<int>(m - row) : ROWS) : 0;
        const bool whole = vecC != 0 && nrows == ROWS;
        double *out = C + row + j * ldc;
        double2 old[ROWS / 2];
#pragma unroll
        for (int h = 0; h < ROWS / 2; ++h) old[h] = make_double2(0.0, 0.0);
        if (whole && beta != 0.0) {
#pragma unroll
            for (int h = 0; h < ROWS / 2; ++h) old[h] = *reinterpret_cast<const double2 *>(out + 2 * h);
        }
        const int sb = valid ? shiftB[j] : 0;
        int sa[ROWS];
#pragma unroll
        for (int h = 0; h < ROWS; ++h) sa[h] = h < nrows ? shiftA[row + h] : 0;

        // ---- this thread's ROWS outputs as rows t of the ROWS operand tiles
#pragma unroll
        for (int h = 0; h < ROWS; ++h) {
            uint32_t kw[8];
            if constexpr (RB == 2) {
                // K = 2 i + a: the two bytes of modulus i; word q holds moduli 2q, 2q+1
#pragma unroll
                for (int q = 0; q < 8; ++q) kw[q] = __byte_perm(w[2 * q], w[2 * q + 1], h ? 0x7632 : 0x5410);
            } else {
                // K = i: byte h of every modulus' word; word q holds moduli 4q .. 4q+3
                const uint32_t sel = static_cast<uint32_t>(((4 + h) << 4) | h);
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    kw[q] = __byte_perm(__byte_perm(w[4 * q], w[4 * q + 1], sel), __byte_perm(w[4 * q + 2], w[4 * q + 3], sel), 0x5410);
#pragma unroll
                for (int q = 4; q < 8; ++q) kw[q] = 0u;
            }
            unsigned char *rowp = &tileA[h][(t >> 3) * 256 + (t & 7) * 16];
            *reinterpret_cast<uint4 *>(rowp) = make_uint4(kw[0], kw[1], kw[2], kw[3]);
            *reinterpret_cast<uint4 *>(rowp + 128) = make_uint4(kw[4], kw[5], kw[6], kw[7]);
        }
        // the tensor core reads shared memory through the asynchronous proxy
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (t == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int h = 0; h < ROWS; ++h)
                mma_u8(tmem_base + 16u * h, plain_desc(smem_addr(tileA[h]), 128, 256), descB);
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
        }
        // bounded wait for the products
        bool ok = false;
#pragma unroll 1
        for (int it = 0; it < 4096 && !ok; ++it) ok = bar_try_wait(bar, phase);
        if (!ok) {
            const unsigned long long start = timer_ns();
            while (!ok && timer_ns() - start < 2000000000ull) {
#pragma unroll 1
                for (int it = 0; it < 256 && !ok; ++it) ok = bar_try_wait(bar, phase);
            }
        }
        if (__syncthreads_or(ok ? 0 : 1)) {              // block-uniform outcome
            if (t == 0) atomicOr(status, 1u << OZ_ERR_TIMEOUT);
            alive = false;
            break;
        }
        phase ^= 1u;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

        const double nan = __longlong_as_double(0x7FF8000000000000ll);
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
        double val[ROWS];
#pragma unroll
        for (int h = 0; h < ROWS; ++h) {
            uint32_t P[16];
            tmem_ld16(lane_addr + 16u * h, P);
            const bool bad = sb == OZ_NONFINITE_SHIFT || sa[h] == OZ_NONFINITE_SHIFT;
            val[h] = (bad ? nan : finish_from_sums<SET>(P, sa[h] + sb)) * alpha;
        }
        if (whole) {
#pragma unroll
            for (int h = 0; h < ROWS / 2; ++h)
                *reinterpret_cast<double2 *>(out + 2 * h) = make_double2(old[h].x + val[2 * h], old[h].y + val[2 * h + 1]);
        } else {
#pragma unroll
            for (int h = 0; h < ROWS; ++h)
                if (h < nrows) out[h] = beta != 0.0 ? out[h] + val[h] : val[h];
        }
        // the next step's products overwrite the accumulators: every thread has read its rows
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

}  // namespace

oz_status_t upload_hosted_constants()
{
    static HostedConst host[kNumSets];
    for (int set = 0; set < kNumSets; ++set) {
        HostedConst &K = host[set];
        unsigned __int128 M = 1;
        for (int i = 0; i < set_r(set); ++i) M *= static_cast<unsigned>(modulus(set, i));
        for (int s = 0; s < 16; ++s)
            for (int kb = 0; kb < 32; ++kb) K.B[s][kb] = 0;
        const int rb = residue_bytes(set);
        unsigned long long cmax_sum = 0;                   // sum of the largest stored residues
        for (int i = 0; i < set_r(set); ++i) {
            const unsigned mi = static_cast<unsigned>(modulus(set, i));
            const unsigned __int128 W = M / mi;
            const unsigned wm = static_cast<unsigned>(W % mi);
            unsigned inv = 0;
            for (unsigned c = 1; c < mi; ++c)
                if ((static_cast<unsigned long long>(wm) * c) % mi == 1) { inv = c; break; }
            const unsigned __int128 V = W * inv;           // < M
            for (int b = 0; b < 16; ++b) {
                const unsigned char byte = static_cast<unsigned char>(V >> (8 * b));
                for (int a = 0; a < rb; ++a) {
                    const int s = a + b, kidx = rb == 2 ? 2 * i + a : i;
                    if (s < 16) K.B[s][kidx] = byte;
                    else if (byte) return OZ_ERR_UNSUPPORTED;     // would need a seventeenth position
                }
            }
            cmax_sum += rb == 2 ? 2 * mi : mi;             // two-byte sets store a representative below 2 m_i
        }
        for (int i = 0; i < 4; ++i) {
            K.M[i] = static_cast<uint32_t>(M >> (32 * i));
            K.Mh[i] = static_cast<uint32_t>((M >> 1) >> (32 * i));
        }
        // S < cmax_sum * M: leading bits so that S >> top_shift < 2^30
        int bits = 0;
        for (unsigned __int128 v = static_cast<unsigned __int128>(cmax_sum) * (M >> 64); v; v >>= 1) ++bits;
        bits += 64 + 1;
        K.top_shift = bits - 30 < 96 ? 96 : bits - 30;
        // 2^top_shift / M, rounded down with a margin of 2^-20
        const double scale = ldexp(1.0, K.top_shift - 64) / (static_cast<double>(static_cast<unsigned long long>(M >> 64)) + 1.0);
        K.kappa_scale = static_cast<float>(scale * (1.0 - 1.0 / (1 << 20)));
    }
    OZ_CUDA_CHECK(cudaMemcpyToSymbol(c_hosted, host, sizeof(host)));
    return OZ_OK;
}

oz_status_t launch_reconstruct_hosted(int64_t m, int64_t n, const void *R, const int32_t *shiftA,
                                      const int32_t *shiftB, int set, double alpha, double beta,
                                      double *C, int64_t ldc, int64_t col0, int64_t col1,
                                      cudaStream_t stream)
{
    if (col1 <= col0) return OZ_OK;
    const ResidueTiling t = residue_tiling(m, n, set);
    const int tn0 = static_cast<int>(col0 / t.tile_cols);
    const int ntn = static_cast<int>((col1 + t.tile_cols - 1) / t.tile_cols) - tn0;
    const int vecC = ((ldc & 1) == 0 && (reinterpret_cast<uintptr_t>(C) & 15u) == 0) ? 1 : 0;
    int dev = 0, sms = 148;
    OZ_CUDA_CHECK(cudaGetDevice(&dev));
    OZ_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const int pieces = 64 * 32 * residue_bytes(set) / 4 / 128;
    const int64_t total = static_cast<int64_t>(t.tiles_m) * ntn * t.cg * 16 * pieces;
    // persistent blocks: TMEM (512 columns per SM) admits 16 blocks of 32 columns, 8 of 64
    const int per_sm = residue_bytes(set) == 2 ? 12 : 8;
    const int64_t cap = static_cast<int64_t>(sms) * per_sm;
    const unsigned grid = static_cast<unsigned>(total < cap ? total : cap);
    unsigned int *status = device_status_word();
#define OZ_RECON_HOSTED(SET_)                                                                               \
    reconstruct_hosted_kernel<SET_><<<grid, 128, 0, stream>>>(R, t.cg, t.tiles_n, tn0, ntn, t.tiles_m, m, n, col0, \
                                                              col1, shiftA, shiftB, alpha, beta, C, ldc, vecC, status)
    if (set == 2) OZ_RECON_HOSTED(2);
    else if (set == 0) OZ_RECON_HOSTED(0);
    else OZ_RECON_HOSTED(1);
#undef OZ_RECON_HOSTED
    count_launch();
    OZ_CUDA_CHECK(cudaGetLastError());
    return OZ_OK;
}

}  // namespace oz
