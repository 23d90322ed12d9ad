// Fused mode of the residue products for tall-skinny shapes (Sec. "Storage Modes", mode F; "O4:
// pipelining"): the planes of A are never written to memory.  The kernel reads FP64 A and the shifts
// of its rows, converts each tile of A into plane bytes inside the shared-memory ring that feeds the
// tensor core (quantise -> limbs -> residues -> table look-up, the same arithmetic as the
// deconstruction kernels), and multiplies it with B's planes, which are materialised as always and
// stream from L2.  Included by oz_gemm_sm100.cu inside its anonymous namespace.
//
// Geometry.  n <= 128: all lines of B are the M = 128 lanes of one accumulator.  A tile of 64 lines of
// A is the N dimension, so an accumulator takes 64 TMEM columns and the 512 columns hold the two
// accumulators (merged schedule) of FOUR moduli.  A work item is (tile of 64 rows); it is processed
// in passes of four moduli (lambda_A = r / 4 re-reads and re-quantisations of the tile, the paper's
// modulus blocking n_blk = 4), each pass a K-loop over stages of 32 inner indices:
//   warp 0        TMA producer: for every plane of the pass, the two 16-byte K halves of 128 lines of
//                 B (un-swizzled core-matrix layout: 8 rows x 16 bytes contiguous)
//   warp 1        MMA issuer: per stage three tcgen05.mma (M 128, N 64, K 32) per modulus
//   warps 2..5    epilogue, once per pass: drain the eight accumulators, combine, reduce modulo m_i,
//                 store canonical residues in the public layout R[mod][j][ldr]
//   warps 6..21   converters: thread (row, 4 consecutive inner indices) loads four doubles, makes the
//                 limbs once and writes 4 bytes of every plane of the pass's moduli into the stage
// The ring has two stages of 72 KiB (A part 24 KiB, B part 48 KiB) beside the look-up table.
// Exactness needs one accumulator per job over the whole K (no K segments): the host takes this
// mode only for k within the exact depth of the merged accumulator.
//
// Every wait is bounded like in residue_gemm_kernel; on expiry the CTA records OZ_ERR_TIMEOUT,
// leaves its loops, frees TMEM and returns.

constexpr int F_LINES = 64;                         // rows of A per tile = accumulator columns
constexpr int F_K = 32;                             // inner indices per stage
constexpr int F_GROUP = 4;                          // moduli per pass
constexpr int F_MAXP = 3 * F_GROUP;                 // planes per stage at most
constexpr int F_A_PLANE = 2 * F_LINES * 16;         // bytes of one A plane in a stage: [K half][row][16]
constexpr int F_B_PLANE = 2 * 128 * 16;             // bytes of one B plane in a stage
constexpr int F_A_BYTES = F_MAXP * F_A_PLANE;       // 24 KiB
constexpr int F_B_BYTES = F_MAXP * F_B_PLANE;       // 48 KiB
constexpr int F_STAGE = F_A_BYTES + F_B_BYTES;
constexpr int F_STAGES = 2;
constexpr int F_CONV_WARPS = 16;
constexpr int F_FIRST_CONV = 6;
constexpr int F_THREADS = (F_FIRST_CONV + F_CONV_WARPS) * 32;     // 704
static_assert(F_CONV_WARPS * 32 * 4 == F_LINES * F_K, "one quad of inner indices per converter thread and stage");

struct FusedGemmParams {
    const double *A;                // FP64 operand, column-major m x k
    int64_t lda;
    const int32_t *shiftA;
    const uint32_t *lut_global;     // plane table of (set, substrate)
    int tz;
    int tiles;                      // tiles of 64 rows
    int passes;                     // groups of four moduli
    int nks;                        // stages per pass = ceil(k / 32)
};

__host__ __device__ constexpr size_t fused_gemm_smem(int set)
{
    return static_cast<size_t>(lut_words(set)) * 4 + F_STAGES * F_STAGE + 1024 /*alignment*/ + 256 /*barriers*/;
}

// shared-memory matrix descriptor, K-major, no swizzle: core matrices of 8 rows x 16 bytes (128
// contiguous bytes); `lbo`: bytes to the core matrix next in K, `sbo`: bytes to the next 8-row group
__device__ __forceinline__ uint64_t plain_smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((addr >> 4) & 0x3FFFu);
    d |= static_cast<uint64_t>((lbo >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>((sbo >> 4) & 0x3FFFu) << 32;
    d |= static_cast<uint64_t>(1) << 46;                 // descriptor version of sm_100
    return d;                                            // bits 61..63 = 0: no swizzle
}

template <int SUB>
__host__ __device__ constexpr uint32_t fused_instr_desc()
{
    uint32_t cfmt = SUB == 0 ? 1u /*f32*/ : 2u /*s32*/;
    uint32_t abfmt = SUB == 0 ? 0u /*e4m3*/ : 1u /*s8*/;
    return (cfmt << 4) | (abfmt << 7) | (abfmt << 10) | (static_cast<uint32_t>(F_LINES >> 3) << 17) |
           (static_cast<uint32_t>(BLOCK_M >> 4) << 24);
}

// planes of the moduli 4G .. 4G+3 of the set for one quad of elements, written at their position
// inside the stage (plane index relative to the first plane of the pass)
template <int SET, int LAYOUT, int G, int... S>
__device__ __forceinline__ void convert_pass_moduli(std::integer_sequence<int, S...>, const uint32_t (&l0)[4],
                                                    const uint32_t (&l1)[4], const uint32_t (&l2)[4],
                                                    const uint32_t (&l3)[4], const uint32_t *lut, uint8_t *out)
{
    constexpr int first = first_plane(SET, F_GROUP * G, LAYOUT);
    (convert_modulus<SET, LAYOUT, F_GROUP * G + S>(l0, l1, l2, l3, lut, out - first * F_A_PLANE, F_A_PLANE), ...);
}

template <int SET, int LAYOUT, int G>
__device__ __forceinline__ void convert_pass(const uint32_t (&l0)[4], const uint32_t (&l1)[4],
                                             const uint32_t (&l2)[4], const uint32_t (&l3)[4],
                                             const uint32_t *lut, uint8_t *out)
{
    constexpr int left = set_r(SET) - F_GROUP * G;
    constexpr int count = left < F_GROUP ? (left > 0 ? left : 0) : F_GROUP;
    convert_pass_moduli<SET, LAYOUT, G>(std::make_integer_sequence<int, count>{}, l0, l1, l2, l3, lut, out);
}

template <int SUB, int SET, int LAYOUT_A>
__global__ void __launch_bounds__(F_THREADS, 1)
fused_gemm_kernel(const __grid_constant__ CUtensorMap mapB, const __grid_constant__ GemmParams p,
                  const __grid_constant__ FusedGemmParams f)
{
    constexpr int RB = residue_bytes(SET);
    constexpr int LUT_BYTES = lut_words(SET) * 4;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;                      // 1024-byte aligned ring
    unsigned char *ring_gen = smem_raw + (ring - raw);
    const uint32_t lut_addr = ring + F_STAGES * F_STAGE;
    uint32_t *lut = reinterpret_cast<uint32_t *>(ring_gen + F_STAGES * F_STAGE);
    const uint32_t bars = lut_addr + LUT_BYTES;
    const uint32_t full_bar = bars;                                    // F_STAGES x 8 bytes
    const uint32_t empty_bar = bars + 8 * F_STAGES;
    const uint32_t tfull_bar = bars + 16 * F_STAGES;
    const uint32_t tempty_bar = tfull_bar + 8;
    const uint32_t tmem_slot = tempty_bar + 8;
    unsigned char *bar_gen = ring_gen + F_STAGES * F_STAGE + LUT_BYTES;
    volatile uint32_t *tmem_base_ptr = reinterpret_cast<volatile uint32_t *>(bar_gen + 16 * F_STAGES + 16);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bar_gen + 16 * F_STAGES + 24);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    for (int i = threadIdx.x; i < lut_words(SET); i += F_THREADS) lut[i] = f.lut_global[i];
    if (threadIdx.x == 0) {
        for (int s = 0; s < F_STAGES; ++s) {
            mbar_init(full_bar + 8 * s, 1 + F_CONV_WARPS);     // the producer's expect_tx arrive + one per converter warp
            mbar_init(empty_bar + 8 * s, 1);
        }
        mbar_init(tfull_bar, 1);
        mbar_init(tempty_bar, 4);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc<1>(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_base_ptr;

    // planes of pass g: [first, first + count) in both operands' plane order (same counts on both sides)
    auto pass_first_plane = [&](int g) { return p.mod[g * F_GROUP].planeA0; };
    auto pass_moduli = [&](int g) { return min(F_GROUP, p.r - g * F_GROUP); };
    auto pass_planes = [&](int g) {
        const int last = g * F_GROUP + pass_moduli(g) - 1;
        return p.mod[last].planeA0 + (p.mod[last].kind == 0 ? 2 : 3) - p.mod[g * F_GROUP].planeA0;
    };

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------------------ TMA producer: B's planes
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && !p.stall_producer && tile < f.tiles; tile += gridDim.x)
                for (int g = 0; ok && g < f.passes; ++g) {
                    const int np = pass_planes(g), firstB = p.mod[g * F_GROUP].planeB0;
                    for (int ks = 0; ks < f.nks; ++ks) {
                        ok = mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag, p.status);
                        if (!ok) break;
                        const uint32_t fb = full_bar + 8 * stage;
                        const uint32_t sb = ring + stage * F_STAGE + F_A_BYTES;
                        mbar_expect_tx(fb, static_cast<uint32_t>(np) * F_B_PLANE);
                        for (int lp = 0; lp < np; ++lp) {
                            tma_load_3d(sb + lp * F_B_PLANE, &mapB, fb, ks * F_K, 0, firstB + lp);
                            tma_load_3d(sb + lp * F_B_PLANE + F_B_PLANE / 2, &mapB, fb, ks * F_K + 16, 0, firstB + lp);
                        }
                        if (++stage == F_STAGES) { stage = 0; phase ^= 1u; }
                    }
                }
            if (!ok) {
                unsigned long long t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 2000000ull) { }     // copies in flight get a bounded time to land
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ------------------------------------------------------------ MMA issuer
            constexpr uint32_t idesc = fused_instr_desc<SUB>();
            int stage = 0;
            uint32_t phase = 0, tphase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < f.tiles; tile += gridDim.x)
                for (int g = 0; ok && g < f.passes; ++g) {
                    // the accumulators are free once the epilogue of the previous pass has read them
                    ok = mbar_wait(tempty_bar, tphase ^ 1u, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
                    const int nm = pass_moduli(g), first = pass_first_plane(g);
                    for (int ks = 0; ks < f.nks; ++ks) {
                        ok = mbar_wait(full_bar + 8 * stage, phase, abort_flag, p.status);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t sa = ring + stage * F_STAGE, sb = sa + F_A_BYTES;
                        for (int s = 0; s < nm; ++s) {
                            const ModInfo &mi = p.mod[g * F_GROUP + s];
                            for (int job = 0; job < 2; ++job) {
                                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(s * 2 * F_LINES + job * F_LINES);
                                const int npairs = job_pairs(mi, job);
                                for (int pair = 0; pair < npairs; ++pair) {
                                    int pa, pb;
                                    job_planes(mi, job, pair, &pa, &pb);
                                    const uint64_t dm = plain_smem_desc(sb + (pb - mi.planeB0 + mi.planeA0 - first) * F_B_PLANE,
                                                                        F_B_PLANE / 2, 128);
                                    const uint64_t dn = plain_smem_desc(sa + (pa - first) * F_A_PLANE, F_A_PLANE / 2, 128);
                                    umma<SUB, 1>(d_tmem, dm, dn, idesc, (ks > 0 || pair > 0) ? 1u : 0u);
                                }
                            }
                        }
                        umma_commit<1>(empty_bar + 8 * stage);
                        if (++stage == F_STAGES) { stage = 0; phase ^= 1u; }
                    }
                    if (!ok) break;
                    umma_commit<1>(tfull_bar);
                    tphase ^= 1u;
                }
            if (!ok) {
                unsigned long long t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 2000000ull) { }
            }
        }
    } else if (warp < F_FIRST_CONV) {
        // ---------------------------------------------------------------- epilogue, once per pass
        const int q = warp & 3;                                  // TMEM lane quarter this warp may read
        const int64_t j = q * 32 + lane;                         // column of C = line of B
        uint32_t tphase = 0;
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < f.tiles; tile += gridDim.x)
            for (int g = 0; ok && g < f.passes; ++g) {
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(tfull_bar, tphase, abort_flag, p.status));
                if (!ok) break;
                tc_fence_after();
                const int nm = pass_moduli(g);
                const int64_t i0 = static_cast<int64_t>(tile) * F_LINES;
                for (int s = 0; s < nm; ++s) {
                    const int mod = g * F_GROUP + s;
                    const ModInfo &mi = p.mod[mod];
                    const float mm = mi.m, inv_m = mi.inv_m;
                    const uint32_t im = mi.mi, imagic = mi.magic, ibias = mi.bias;
#pragma unroll 1
                    for (int half = 0; half < 2; ++half) {
                        uint32_t comb[32];
#pragma unroll
                        for (int c = 0; c < 32; ++c) comb[c] = 0u;
#pragma unroll
                        for (int job = 0; job < 2; ++job) {
                            const float wj = mi.w[job];
                            const int iwj = mi.iw[job];
                            const bool reduce_first = mi.reduce[job] != 0;
                            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                                   static_cast<uint32_t>(s * 2 * F_LINES + job * F_LINES + half * 32);
#pragma unroll
                            for (int c0 = 0; c0 < 32; c0 += 16) {
                                uint32_t v[16];
                                tmem_ld16(taddr + c0, v);
#pragma unroll
                                for (int e = 0; e < 16; ++e) {
                                    if constexpr (SUB == 0) {
                                        float acc = __uint_as_float(v[e]);
                                        if (reduce_first) {
                                            const float quot = fmaf(acc, inv_m, 12582912.0f) - 12582912.0f;
                                            acc = fmaf(-quot, mm, acc);
                                        }
                                        comb[c0 + e] = __float_as_uint(fmaf(acc, wj, __uint_as_float(comb[c0 + e])));
                                    } else {
                                        int acc = static_cast<int>(v[e]);
                                        if (reduce_first) {
                                            uint32_t u = v[e] + ibias;
                                            uint32_t r = u - __umulhi(u, imagic) * im;
                                            acc = static_cast<int>(min(r, r - im));
                                        }
                                        comb[c0 + e] = static_cast<uint32_t>(acc * iwj + static_cast<int>(comb[c0 + e]));
                                    }
                                }
                            }
                        }
                        // canonical residues of rows i0 + half*32 .. +31 of column j, packed RB bytes each
                        uint32_t packed[32 * RB / 4];
#pragma unroll
                        for (int c = 0; c < 32; c += 4 / RB) {
                            uint32_t b[4 / RB];
#pragma unroll
                            for (int e = 0; e < 4 / RB; ++e) {
                                if constexpr (SUB == 0) {
                                    const float t = __uint_as_float(comb[c + e]);
                                    const float quot = fmaf(t, inv_m, 12582912.0f) - 12582912.0f;
                                    float res = fmaf(-quot, mm, t);
                                    res = res < 0.0f ? res + mm : res;
                                    b[e] = __float_as_uint(res + 8388608.0f) & 0xFFFFu;
                                } else {
                                    const uint32_t u = comb[c + e] + ibias;
                                    const uint32_t r = u - __umulhi(u, imagic) * im;
                                    b[e] = min(r, r - im);
                                }
                            }
                            if constexpr (RB == 2) packed[c / 2] = b[0] | (b[1] << 16);
                            else packed[c / 4] = b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24);
                        }
                        if (j < p.n) {
                            // ldr is a multiple of 64 and the tile starts on a multiple of 64: 16-byte aligned
                            unsigned char *dst = static_cast<unsigned char *>(p.R) +
                                                 (static_cast<int64_t>(mod) * p.mod_stride + j * p.ldr + i0 + half * 32) * RB;
#pragma unroll
                            for (int c = 0; c < 32 * RB / 16; ++c)
                                *reinterpret_cast<uint4 *>(dst + 16 * c) =
                                    make_uint4(packed[4 * c], packed[4 * c + 1], packed[4 * c + 2], packed[4 * c + 3]);
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_relaxed(tempty_bar);
                tphase ^= 1u;
            }
    } else {
        // ---------------------------------------------------------------- converters: A's planes
        // thread -> (row r of the tile, K half h, quad kq of four inner indices): four consecutive lanes
        // fill one 16-byte row chunk, a warp 128 contiguous bytes of every plane (no bank conflicts)
        const int ct = threadIdx.x - F_FIRST_CONV * 32;
        const int kq = ct & 3, r = (ct >> 2) & (F_LINES - 1), h = ct >> 8;
        const bool tz = f.tz != 0;
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < f.tiles; tile += gridDim.x) {
            const int64_t row = static_cast<int64_t>(tile) * F_LINES + r;
            const int sigma_raw = row < p.m ? f.shiftA[row] : OZ_NONFINITE_SHIFT;
            const bool dead = sigma_raw == OZ_NONFINITE_SHIFT;     // beyond m, or a row with Inf/NaN: zero planes
            const int sigma = dead ? 0 : sigma_raw;
            const int koff = h * 16 + kq * 4;
            const double *src = f.A + (dead ? 0 : row) + static_cast<int64_t>(koff) * f.lda;
            for (int g = 0; ok && g < f.passes; ++g) {
                double x[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) x[e] = (!dead && koff + e < p.k) ? src[e * f.lda] : 0.0;
                for (int ks = 0; ks < f.nks; ++ks) {
                    // the next stage's elements are requested before this stage's arithmetic
                    double xn[4];
                    const int64_t kn = static_cast<int64_t>(ks + 1) * F_K + koff;
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        xn[e] = (!dead && ks + 1 < f.nks && kn + e < p.k) ? src[(static_cast<int64_t>(ks + 1) * F_K + e) * f.lda] : 0.0;
                    uint32_t l0[4], l1[4], l2[4], l3[4];
                    split_limbs4(x, sigma, tz, l0, l1, l2, l3);
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag, p.status));
                    if (!ok) break;
                    uint8_t *out = ring_gen + stage * F_STAGE + (h * F_LINES + r) * 16 + kq * 4;
                    switch (g) {
                    case 0: convert_pass<SET, LAYOUT_A, 0>(l0, l1, l2, l3, lut, out); break;
                    case 1: convert_pass<SET, LAYOUT_A, 1>(l0, l1, l2, l3, lut, out); break;
                    case 2: convert_pass<SET, LAYOUT_A, 2>(l0, l1, l2, l3, lut, out); break;
                    default: convert_pass<SET, LAYOUT_A, 3>(l0, l1, l2, l3, lut, out); break;
                    }
                    // the tensor core reads shared memory through the asynchronous proxy
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0)
                        asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0];" ::"r"(full_bar + 8 * stage) : "memory");
                    if (++stage == F_STAGES) { stage = 0; phase ^= 1u; }
#pragma unroll
                    for (int e = 0; e < 4; ++e) x[e] = xn[e];
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<1>(tmem_base, TMEM_COLS);
    }
}
