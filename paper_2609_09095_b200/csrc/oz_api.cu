// C-ABI entry points of liboz_b200.so: argument checks, per-device set-up, workspace carving
// and the oz_dgemm driver (Algorithm 1 reduced to materialised planes and three stages).
#include <atomic>
#include <cmath>
#include <mutex>

#include "oz_internal.h"

namespace oz {

// ------------------------------------------------------------------------------------------
// per-device objects: plane lookup tables and the sticky status word
// ------------------------------------------------------------------------------------------
__device__ uint32_t g_lut[kNumSets][3][kLutWords];
// status block: [0] sticky condition bits; [1], [2] smallest flatness code of the lines of A / B seen
// since the last query (exponent-span check); [3] the threshold of the modulus set last used
__device__ unsigned int g_status[5];
const unsigned int kStatusReset[5] = {0u, 0xFFFFFFFFu, 0xFFFFFFFFu, 0u, 0u};

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
bool g_ready[kMaxDevices] = {};
const uint32_t *g_lut_addr[kMaxDevices] = {};
unsigned int *g_status_addr[kMaxDevices] = {};
// side stream on which the whole-method calls deconstruct B while A is deconstructed on the caller's
cudaStream_t g_side_stream[kMaxDevices] = {};
cudaEvent_t g_fork[kMaxDevices] = {}, g_join[kMaxDevices] = {};
void *g_workspace[kMaxDevices] = {};
size_t g_workspace_bytes[kMaxDevices] = {};
std::atomic<uint64_t> g_launches{0};
// per-stage timing hook: one set of five caller-owned events per device
cudaEvent_t g_stage_events[kMaxDevices][5] = {};
bool g_stage_events_on[kMaxDevices] = {};

// the workspace registered for a device (read under the mutex that oz_set_workspace writes it under)
void registered_workspace(int dev, char **ws, size_t *bytes)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    *ws = static_cast<char *>(g_workspace[dev]);
    *bytes = g_workspace_bytes[dev];
}

// Is the integer v exactly representable in E4M3 (the set of Lemma 1)?  If so return its
// byte code through *code.  OCP E4M3: bias 7, 3 mantissa bits, largest finite value 448.
bool e4m3_code(int v, int *code)
{
    if (v == 0) { *code = 0; return true; }
    int a = v < 0 ? -v : v;
    if (a > 448) return false;
    int e = 0;
    while ((2 << e) <= a) ++e;              // e = floor(log2 a)
    int scaled = a << 3;                     // a * 8
    if (scaled % (1 << e) != 0) return false;
    int mant = (scaled >> e) - 8;            // 0..7
    *code = ((v < 0) ? 0x80 : 0) | ((e + 7) << 3) | mant;
    return true;
}

int floor_mod(int a, int b) { int r = a % b; return r < 0 ? r + b : r; }

// Packed plane bytes of the canonical residue u of modulus m (Algorithm 2, split lines):
// byte 0 = d0, byte 1 = d1, byte 2 = d0+d1 (zero for a square modulus).
uint32_t lut_entry(int u, int m, int substrate)
{
    int d = (2 * u >= m) ? u - m : u;        // centred, -m/2 included
    if (substrate == 2) return static_cast<uint32_t>(d & 0xFF);   // native INT8: the residue is the operand
    int s = square_root(m);
    int dig[3] = {0, 0, 0};
    if (s) {
        int half = s / 2;
        dig[0] = floor_mod(d + half, s) - half;
        dig[1] = (d - dig[0]) / s;
    } else {
        dig[0] = floor_mod(d + 8, 16) - 8;
        dig[1] = (d - dig[0]) / 16;
        int code;
        if (!e4m3_code(dig[0] + dig[1], &code)) {        // Lemma 1: one predicated carry
            int sg = (dig[0] > 0) - (dig[0] < 0);
            dig[0] -= 16 * sg;
            dig[1] += sg;
        }
        dig[2] = dig[0] + dig[1];
    }
    uint32_t word = 0;
    for (int q = 0; q < 3; ++q) {
        int byte = 0;
        if (substrate == 0) e4m3_code(dig[q], &byte);
        else byte = dig[q] & 0xFF;
        word |= static_cast<uint32_t>(byte) << (8 * q);
    }
    if (!s) {                                // byte 3: what the merged schedule swaps in
        int byte = 0;
        if (substrate == 0) e4m3_code(-16 * dig[1], &byte);   // FP8: the pre-scaled plane -16*d1
        else byte = (-dig[0]) & 0xFF;                          // INT8: -d0 (4*d1 is a shift of byte 1)
        word |= static_cast<uint32_t>(byte) << 24;
    }
    return word;
}

unsigned __int128 set_product(int set)
{
    unsigned __int128 M = 1;
    for (int i = 0; i < set_r(set); ++i) M *= static_cast<unsigned>(modulus(set, i));
    return M;
}

uint64_t isqrt_u128(unsigned __int128 v)
{
    uint64_t r = static_cast<uint64_t>(sqrtl(static_cast<long double>(v)));
    while (static_cast<unsigned __int128>(r) * r > v) --r;
    while (static_cast<unsigned __int128>(r + 1) * (r + 1) <= v) ++r;
    return r;
}

}  // namespace

bool decode_route(uint32_t route, Route *out)
{
    uint32_t sub = route & 0x00Fu, q = route & 0x0F0u, sc = route & 0xF00u, ac = route & 0x3000u;
    if (route & ~0x1FFFFu) return false;
    out->hosted = (route & OZ_RECON_TENSOR) != 0;
    out->fallback = (route & OZ_FALLBACK_FP64) != 0;
    out->fused = (route & OZ_STORAGE_FUSED) != 0;
    if (ac == 0) out->acc = 0;
    else if (ac == OZ_ACC_MERGED) out->acc = 1;
    else if (ac == OZ_ACC_SEPARATE) out->acc = 2;
    else return false;
    if (sub == 0 || sub == OZ_SUB_FP8) out->substrate = 0;
    else if (sub == OZ_SUB_INT8) out->substrate = 1;
    else if (sub == OZ_SUB_INT8_NATIVE) out->substrate = 2;
    else return false;
    if (q == 0 || q == OZ_QUANT_RN) out->quant = 0;
    else if (q == OZ_QUANT_TZ) out->quant = 1;
    else return false;
    if (sc == 0 || sc == OZ_SCALE_CS) out->rule = 1;
    else if (sc == OZ_SCALE_MAXEXP) out->rule = 0;
    else if (sc == OZ_SCALE_ACCURATE) out->rule = 2;
    else return false;
    return true;
}

// the native INT8 route needs every centred residue to fit a signed byte: all-byte set A only
bool decode_route_for_set(int set, uint32_t route, Route *out)
{
    if (!decode_route(route, out)) return false;
    if (out->merged() && out->native()) return false;         // one plane per modulus: nothing to merge
    return !(out->native() && set != OZ_SET_A);
}

// Fixes the accumulator schedule of a call.  `automatic`: the whole-method entry points, whose
// planes are internal, take the merged schedule on the digit substrates (one accumulator drain fewer
// per non-square modulus at no extra plane; the GEMM cuts a long k into segments that each stay exact);
// the stage entry points default to separate accumulators because what their d1 plane holds is part
// of the interface.
oz_status_t resolve_schedule(int set, int64_t k, int64_t n, bool automatic, Route *rt)
{
    if (rt->acc == 0)
        rt->acc = (automatic && !rt->native() && k > 0) ? 1 : 2;
    return OZ_OK;
}

void budget_maxexp(int set, int64_t k, int *tA, int *tB)
{
    unsigned __int128 v = (set_product(set) - 1) / 2 / static_cast<unsigned __int128>(k > 0 ? k : 1);
    int T = -1;
    while (v) { ++T; v >>= 1; }
    *tB = T / 2;
    *tA = T - T / 2;
}

// floor(log2 H') of the accurate rule: H' = floor(((M-1)/2) / 129) * 128
int accurate_budget_log2(int set)
{
    unsigned __int128 v = ((set_product(set) - 1) / 2 / 129) * 128;
    int L = -1;
    while (v) { ++L; v >>= 1; }
    return L;
}

// Exponent-span check: a call is flagged when  qA qB < floor(floor(2^120 / 3) / (((M-1)/2) >> 20)),
// i.e. phiA^2 phiB^2 < (16/3) 2^104 / ((M-1)/2), with q = floor(2^16 phi^2) the smallest flatness of an
// operand's lines (see scan_finalize_kernel).
unsigned int esc_threshold(int set)
{
    unsigned __int128 H = (set_product(set) - 1) / 2;
    unsigned __int128 t = ((static_cast<unsigned __int128>(1) << 120) / 3) / (H >> 20);
    return t > 0xFFFFFFFFu ? 0xFFFFFFFFu : static_cast<unsigned int>(t);
}

void cs_bound_squared(int set, int64_t k, uint64_t *lo, uint64_t *hi)
{
    uint64_t bnd = isqrt_u128((set_product(set) - 1) / 2);
    uint64_t kk = static_cast<uint64_t>(k > 0 ? k : 1);
    uint64_t s = isqrt_u128(kk);
    uint64_t g = (s * s == kk) ? (s + 1) / 2 : s / 2 + 1;   // ceil(sqrt(k)/2)
    unsigned __int128 G = bnd - g;
    unsigned __int128 G2 = G * G;
    *lo = static_cast<uint64_t>(G2);
    *hi = static_cast<uint64_t>(G2 >> 64);
}

oz_status_t ensure_device_ready()
{
    int dev = 0;
    OZ_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return OZ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_ready[dev]) return OZ_OK;
    static uint32_t host_lut[kNumSets][3][kLutWords];
    for (int set = 0; set < kNumSets; ++set)
        for (int sub = 0; sub < 3; ++sub) {
            int off = 0;
            for (int i = 0; i < set_r(set); ++i) {
                int m = modulus(set, i);
                for (int u = 0; u < kLutSpan * m; ++u) host_lut[set][sub][off + u] = lut_entry(u % m, m, sub);
                off += kLutSpan * m;
            }
            for (; off < kLutWords; ++off) host_lut[set][sub][off] = 0;
        }
    OZ_CUDA_CHECK(cudaMemcpyToSymbol(g_lut, host_lut, sizeof(host_lut)));
    OZ_CUDA_CHECK(cudaMemcpyToSymbol(g_status, kStatusReset, sizeof(kStatusReset)));
    void *p = nullptr;
    OZ_CUDA_CHECK(cudaGetSymbolAddress(&p, g_lut));
    g_lut_addr[dev] = static_cast<const uint32_t *>(p);
    OZ_CUDA_CHECK(cudaGetSymbolAddress(&p, g_status));
    g_status_addr[dev] = static_cast<unsigned int *>(p);
    oz_status_t st = upload_reconstruct_constants();
    if (st != OZ_OK) return st;
    unsigned char codes[33];
    for (int d = 0; d <= 32; ++d) {
        int code = 0;
        e4m3_code(d, &code);            // odd digits above 16 are never produced
        codes[d] = static_cast<unsigned char>(code);
    }
    st = upload_bound_codes(codes);
    if (st != OZ_OK) return st;
    st = upload_hosted_constants();
    if (st != OZ_OK) return st;
    g_ready[dev] = true;
    return OZ_OK;
}

// The side stream and its two events exist only for the whole-method calls and are created on a
// device's first such call; the stage entry points (the allocation-free one among them) never get here.
oz_status_t ensure_side_stream(int dev)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_side_stream[dev]) return OZ_OK;
    cudaStream_t st = nullptr;
    OZ_CUDA_CHECK(cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking));
    OZ_CUDA_CHECK(cudaEventCreateWithFlags(&g_fork[dev], cudaEventDisableTiming));
    OZ_CUDA_CHECK(cudaEventCreateWithFlags(&g_join[dev], cudaEventDisableTiming));
    g_side_stream[dev] = st;
    return OZ_OK;
}

const uint32_t *device_lut(int set, int substrate)
{
    int dev = 0;
    cudaGetDevice(&dev);
    return g_lut_addr[dev] + (static_cast<size_t>(set) * 3 + substrate) * kLutWords;
}

unsigned int *device_status_word()
{
    int dev = 0;
    cudaGetDevice(&dev);
    return g_status_addr[dev];
}

void count_launch(int n) { g_launches.fetch_add(static_cast<uint64_t>(n)); }

namespace {

struct Carve {
    size_t off = 0;
    size_t take(size_t bytes)
    {
        size_t at = off;
        off += static_cast<size_t>(round_up(static_cast<int64_t>(bytes), 256));
        return at;
    }
};

// One deconstructed operand: shifts, scan scratch and planes in one caller-owned block.  Used both
// for the call-scoped planes inside the workspace and for the planes that a caller keeps across
// calls (oz_prepare_operand / oz_dgemm_prepared).
struct OperandLayout {
    size_t shift, scratch, planes, total;
    int64_t pitch, stride;
};

OperandLayout operand_layout(int side, int64_t lines, int64_t k, int set, const Route &rt, bool whole_method = false)
{
    OperandLayout o{};
    Carve c;
    o.pitch = round_up(k > 0 ? k : 1, 128);   // whole 128-byte lines per TMA box row (k = 5003 -> 5120)
    o.stride = lines * o.pitch;
    o.shift = c.take(4 * static_cast<size_t>(lines));
    o.scratch = c.take(16 * static_cast<size_t>(lines) + 256);
    // storage mode F keeps no planes of A: they exist only inside the product kernel's shared memory
    o.planes = c.take((whole_method && rt.fused && side == 0) ? 0 : static_cast<size_t>(p_store(set, rt.layout(side))) * o.stride);
    o.total = c.off;
    return o;
}

struct OperandView {
    int32_t *shift;
    void *scratch;
    uint8_t *planes;
    int64_t pitch, stride;
};

OperandView operand_view(char *base, const OperandLayout &o)
{
    return OperandView{reinterpret_cast<int32_t *>(base + o.shift), base + o.scratch,
                       reinterpret_cast<uint8_t *>(base + o.planes), o.pitch, o.stride};
}

size_t residue_bytes_total(int64_t m, int64_t n, int set)
{
    // the tile-ordered private array of the whole-method calls (whole tiles are stored)
    return static_cast<size_t>(round_up(static_cast<int64_t>(residue_bytes(set)) * set_r(set) *
                                        residue_tiling(m, n, set).mod_stride, 256));
}

struct Layout {
    OperandLayout A, B;
    size_t offA, offB, R, total;
    size_t fb_flag, fb_list, fb_count;    // native-path bookkeeping (fallback route only)
};

Layout make_layout(int64_t m, int64_t n, int64_t k, int set, const Route &rt)
{
    Layout L{};
    L.A = operand_layout(0, m, k, set, rt, true);
    L.B = operand_layout(1, n, k, set, rt, true);
    L.offA = 0;
    L.offB = L.A.total;
    L.R = L.offB + L.B.total;
    L.total = L.R + residue_bytes_total(m, n, set);
    if (rt.fallback) {
        L.fb_flag = L.total;
        L.fb_list = L.fb_flag + static_cast<size_t>(round_up(m, 256));
        L.fb_count = L.fb_list + static_cast<size_t>(round_up(4 * m, 256));
        L.total = L.fb_count + 256;
    }
    return L;
}

bool valid_set(int set) { return set == OZ_SET_S || set == OZ_SET_E || set == OZ_SET_A; }

// Optional split of the reconstruction into column panels, used by the host-buffer entry point to
// overlap the transfers of C with the computation: before panel p the stream waits for before[p]
// (when wait_before), after it the stream records after[p].
constexpr int kMaxPanels = 16;
struct PanelPlan {
    int np;
    int64_t col0[kMaxPanels + 1];
    bool wait_before;
    cudaEvent_t *before, *after;
};

// residue GEMMs + reconstruction from two deconstructed operands (stage events [2]..[4])
oz_status_t product_impl(int64_t m, int64_t n, int64_t k, double alpha, const OperandView &a,
                         const OperandView &b, double beta, double *C, int64_t ldc, int set,
                         const Route &rt, cudaStream_t stream, void *R, int dev, const PanelPlan *plan,
                         const unsigned char *skip_rows = nullptr)
{
    const bool ev = g_stage_events_on[dev];
    if (ev) OZ_CUDA_CHECK(cudaEventRecord(g_stage_events[dev][2], stream));
    // the residues stay inside this call: tile-ordered, and the two-byte sets skip the canonicalisation
    oz_status_t st = launch_residue_gemm(m, n, k, a.planes, a.stride, a.pitch, b.planes, b.stride, b.pitch, set,
                                         rt, R, 0, 0, residue_bytes(set) == 2, true, stream);
    if (st != OZ_OK) return st;
    if (ev) OZ_CUDA_CHECK(cudaEventRecord(g_stage_events[dev][3], stream));
    // the CRT recombination: exact FP64 chunk sums on the FP64 pipe, or (OZ_RECON_TENSOR) one small
    // unsigned 8-bit product per 128 outputs on the tensor pipe and an integer tail
    auto reconstruct = [&](int64_t m_, int64_t n_, const void *R_, const int32_t *sa, const int32_t *sb, int set_,
                           double alpha_, double beta_, double *C_, int64_t ldc_, int64_t c0, int64_t c1,
                           cudaStream_t s_) {
        return rt.hosted ? launch_reconstruct_hosted(m_, n_, R_, sa, sb, set_, alpha_, beta_, C_, ldc_, c0, c1, s_)
                         : launch_reconstruct_tiled(m_, n_, R_, sa, sb, set_, alpha_, beta_, C_, ldc_, c0, c1, s_);
    };
    if (skip_rows) {
        st = launch_reconstruct_tiled(m, n, R, a.shift, b.shift, set, alpha, beta, C, ldc, 0, n, stream, skip_rows);
        if (st != OZ_OK) return st;
    } else if (!plan) {
        st = reconstruct(m, n, R, a.shift, b.shift, set, alpha, beta, C, ldc, 0, n, stream);
        if (st != OZ_OK) return st;
    } else {
        for (int p = 0; p < plan->np; ++p) {
            if (plan->wait_before) OZ_CUDA_CHECK(cudaStreamWaitEvent(stream, plan->before[p], 0));
            st = reconstruct(m, n, R, a.shift, b.shift, set, alpha, beta, C, ldc, plan->col0[p],
                             plan->col0[p + 1], stream);
            if (st != OZ_OK) return st;
            OZ_CUDA_CHECK(cudaEventRecord(plan->after[p], stream));
        }
    }
    if (ev) OZ_CUDA_CHECK(cudaEventRecord(g_stage_events[dev][4], stream));
    return OZ_OK;
}

// checks shared by the whole-method entry points; *trivial: nothing (more) to do after k == 0 handling
oz_status_t check_product_args(int64_t m, int64_t n, int64_t k, double alpha, double beta, double *C,
                               int64_t ldc, int set, uint32_t route, cudaStream_t stream, Route *rt,
                               bool *trivial)
{
    *trivial = true;
    if (!valid_set(set) || !decode_route_for_set(set, route, rt)) return OZ_ERR_INVALID_ARG;
    if (m < 0 || n < 0 || k < 0) return OZ_ERR_INVALID_ARG;
    if (!(alpha == 1.0 || alpha == -1.0) || !(beta == 0.0 || beta == 1.0)) return OZ_ERR_UNSUPPORTED;
    if (k > OZ_K_MAX) return OZ_ERR_UNSUPPORTED;
    if (resolve_schedule(set, k, n, true, rt) != OZ_OK) return OZ_ERR_UNSUPPORTED;
    if (m == 0 || n == 0) return OZ_OK;
    if (!C || ldc < m || (reinterpret_cast<uintptr_t>(C) & 7u)) return OZ_ERR_INVALID_ARG;
    if (k == 0) {
        if (beta == 0.0)
            OZ_CUDA_CHECK(cudaMemset2DAsync(C, sizeof(double) * ldc, 0, sizeof(double) * m, n, stream));
        return OZ_OK;
    }
    *trivial = false;
    return OZ_OK;
}

oz_status_t dgemm_impl(int64_t m, int64_t n, int64_t k, double alpha, const double *A, int64_t lda,
                       const double *B, int64_t ldb, double beta, double *C, int64_t ldc, int set,
                       uint32_t route, cudaStream_t stream, char *ws, size_t ws_bytes,
                       const PanelPlan *plan = nullptr)
{
    Route rt;
    bool trivial = true;
    oz_status_t st = check_product_args(m, n, k, alpha, beta, C, ldc, set, route, stream, &rt, &trivial);
    if (st != OZ_OK || trivial) return st;
    if (!A || !B || lda < m || ldb < k || (reinterpret_cast<uintptr_t>(A) & 7u) ||
        (reinterpret_cast<uintptr_t>(B) & 7u))
        return OZ_ERR_INVALID_ARG;
    // out-of-range rows on the native path: defined on the norm scan, FP64 reconstruction, one panel
    if (rt.fallback && (rt.rule != 1 || rt.hosted || plan)) return OZ_ERR_UNSUPPORTED;
    if (rt.fused && rt.rule == 2) return OZ_ERR_UNSUPPORTED;
    Layout L = make_layout(m, n, k, set, rt);
    if (!ws || ws_bytes < L.total) return OZ_ERR_WORKSPACE;
    st = ensure_device_ready();
    if (st != OZ_OK) return st;
    const OperandView a = operand_view(ws + L.offA, L.A), b = operand_view(ws + L.offB, L.B);

    // The two operands are deconstructed side by side: B's chain of short kernels runs on an
    // internal stream that forks from and joins the caller's (their scratch, planes and shifts are
    // disjoint).  Stage event [1] marks the end of A's chain, [2] the join.
    int dev = 0;
    OZ_CUDA_CHECK(cudaGetDevice(&dev));
    st = ensure_side_stream(dev);
    if (st != OZ_OK) return st;
    cudaStream_t side = g_side_stream[dev];
    const bool ev = g_stage_events_on[dev];
    if (ev) OZ_CUDA_CHECK(cudaEventRecord(g_stage_events[dev][0], stream));
    if (rt.rule == 2) {
        // Accurate mode: exponent scans, one magnitude plane per operand (kept in the first plane slot
        // of each operand, which the conversion overwrites afterwards), the bound product on the
        // tensor cores, the shifts from its row and column maxima, then the conversion as usual.
        if (k > kBoundKMax) return OZ_ERR_UNSUPPORTED;
        st = launch_scan(0, m, k, A, lda, set, rt, a.shift, a.scratch, stream);
        if (st == OZ_OK) st = launch_scan(1, n, k, B, ldb, set, rt, b.shift, b.scratch, stream);
        if (st == OZ_OK) st = launch_bound_plane(0, m, k, A, lda, a.scratch, a.planes, a.pitch, stream);
        if (st == OZ_OK) st = launch_bound_plane(1, n, k, B, ldb, b.scratch, b.planes, b.pitch, stream);
        if (st == OZ_OK)
            st = launch_bound_gemm(m, n, k, a.planes, a.pitch, b.planes, b.pitch, bound_maxima(a.scratch, m),
                                   bound_maxima(b.scratch, n), stream);
        const int budget = accurate_budget_log2(set);
        if (st == OZ_OK) st = launch_accurate_finalize(m, a.scratch, budget, a.shift, stream);
        if (st == OZ_OK) st = launch_accurate_finalize(n, b.scratch, budget, b.shift, stream);
        if (st == OZ_OK)
            st = launch_convert_planes(0, m, k, A, lda, set, rt, a.planes, a.stride, a.pitch, a.shift, stream);
        if (ev && st == OZ_OK) OZ_CUDA_CHECK(cudaEventRecord(g_stage_events[dev][1], stream));
        if (st == OZ_OK)
            st = launch_convert_planes(1, n, k, B, ldb, set, rt, b.planes, b.stride, b.pitch, b.shift, stream);
        if (st != OZ_OK) return st;
        return product_impl(m, n, k, alpha, a, b, beta, C, ldc, set, rt, stream, ws + L.R, dev, plan);
    }
    if (rt.fused) {
        // Storage mode F: only the scan of A runs ahead of the product kernel, which converts A's tiles
        // itself; B is deconstructed as always (side stream); residues in the public layout
        if (rt.fallback || rt.hosted || plan || !fused_gemm_applies(m, n, k, set, rt)) return OZ_ERR_UNSUPPORTED;
        OZ_CUDA_CHECK(cudaEventRecord(g_fork[dev], stream));
        OZ_CUDA_CHECK(cudaStreamWaitEvent(side, g_fork[dev], 0));
        st = launch_deconstruct(1, n, k, B, ldb, set, rt, b.planes, b.stride, b.pitch, b.shift, b.scratch, side);
        if (st != OZ_OK) return st;
        OZ_CUDA_CHECK(cudaEventRecord(g_join[dev], side));
        st = launch_scan(0, m, k, A, lda, set, rt, a.shift, a.scratch, stream);
        if (st != OZ_OK) return st;
        if (ev) OZ_CUDA_CHECK(cudaEventRecord(g_stage_events[dev][1], stream));
        OZ_CUDA_CHECK(cudaStreamWaitEvent(stream, g_join[dev], 0));
        if (ev) OZ_CUDA_CHECK(cudaEventRecord(g_stage_events[dev][2], stream));
        const int64_t ldr = round_up(m, 64);
        st = launch_fused_gemm(m, n, k, A, lda, a.shift, b.planes, b.stride, b.pitch, set, rt, ws + L.R, ldr, n * ldr,
                               stream);
        if (st != OZ_OK) return st;
        if (ev) OZ_CUDA_CHECK(cudaEventRecord(g_stage_events[dev][3], stream));
        st = launch_reconstruct(m, n, ws + L.R, ldr, n * ldr, a.shift, b.shift, set, alpha, beta, C, ldc, stream);
        if (st != OZ_OK) return st;
        if (ev) OZ_CUDA_CHECK(cudaEventRecord(g_stage_events[dev][4], stream));
        return OZ_OK;
    }
    OZ_CUDA_CHECK(cudaEventRecord(g_fork[dev], stream));
    OZ_CUDA_CHECK(cudaStreamWaitEvent(side, g_fork[dev], 0));
    st = launch_deconstruct(1, n, k, B, ldb, set, rt, b.planes, b.stride, b.pitch, b.shift, b.scratch, side);
    if (st != OZ_OK) return st;
    OZ_CUDA_CHECK(cudaEventRecord(g_join[dev], side));
    st = launch_deconstruct(0, m, k, A, lda, set, rt, a.planes, a.stride, a.pitch, a.shift, a.scratch, stream);
    if (st != OZ_OK) return st;
    if (ev) OZ_CUDA_CHECK(cudaEventRecord(g_stage_events[dev][1], stream));
    OZ_CUDA_CHECK(cudaStreamWaitEvent(stream, g_join[dev], 0));
    if (!rt.fallback) return product_impl(m, n, k, alpha, a, b, beta, C, ldc, set, rt, stream, ws + L.R, dev, plan);
    // Algorithm 1, last line / Algorithm 3, "ESC range check": the rows that fail the check are left
    // out of the reconstruction and re-issued on the native FP64 path from the caller's old C
    unsigned char *flag = reinterpret_cast<unsigned char *>(ws + L.fb_flag);
    int *list = reinterpret_cast<int *>(ws + L.fb_list);
    unsigned int *count = reinterpret_cast<unsigned int *>(ws + L.fb_count);
    st = launch_esc_rows(a.scratch, m, b.scratch, n, k, set, flag, list, count, stream);
    if (st != OZ_OK) return st;
    st = product_impl(m, n, k, alpha, a, b, beta, C, ldc, set, rt, stream, ws + L.R, dev, nullptr, flag);
    if (st != OZ_OK) return st;
    return launch_native_rows(m, n, k, A, lda, B, ldb, list, count, b.shift, alpha, beta, C, ldc, stream);
}

// Side streams and events of the host-buffer entry point, created once per device.
struct HostPipe {
    bool ready;
    cudaStream_t in, out;
    cudaEvent_t start, ab, done, c[kMaxPanels], r[kMaxPanels];
};
HostPipe g_pipe[kMaxDevices];

oz_status_t ensure_pipe(int dev, HostPipe **out)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    HostPipe &hp = g_pipe[dev];
    if (!hp.ready) {
        OZ_CUDA_CHECK(cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking));
        OZ_CUDA_CHECK(cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking));
        cudaEvent_t *single[3] = {&hp.start, &hp.ab, &hp.done};
        for (cudaEvent_t *e : single) OZ_CUDA_CHECK(cudaEventCreateWithFlags(e, cudaEventDisableTiming));
        for (int p = 0; p < kMaxPanels; ++p) {
            OZ_CUDA_CHECK(cudaEventCreateWithFlags(&hp.c[p], cudaEventDisableTiming));
            OZ_CUDA_CHECK(cudaEventCreateWithFlags(&hp.r[p], cudaEventDisableTiming));
        }
        hp.ready = true;
    }
    *out = &hp;
    return OZ_OK;
}

}  // namespace
}  // namespace oz

using namespace oz;

extern "C" {

oz_status_t oz_set_info(oz_modset_t set, int *r, int *pstore, int *moduli)
{
    if (!valid_set(set)) return OZ_ERR_INVALID_ARG;
    if (r) *r = set_r(set);
    if (pstore) *pstore = p_store(set);
    if (moduli)
        for (int i = 0; i < set_r(set); ++i) moduli[i] = modulus(set, i);
    return OZ_OK;
}

int oz_plane_count(oz_modset_t set, uint32_t route)
{
    Route rt;
    if (!valid_set(set) || !decode_route_for_set(set, route, &rt)) return 0;
    return p_store(set, rt.layout(1));
}

int oz_plane_count_side(oz_modset_t set, uint32_t route, int side)
{
    Route rt;
    if (!valid_set(set) || !decode_route_for_set(set, route, &rt) || (side != 0 && side != 1)) return 0;
    return p_store(set, rt.layout(side));
}

int64_t oz_row_pitch(int64_t k) { return round_up(k > 0 ? k : 1, 16); }

size_t oz_residue_elem_bytes(oz_modset_t set)
{
    return valid_set(set) ? static_cast<size_t>(residue_bytes(set)) : 0;
}

size_t oz_workspace_bytes(int64_t m, int64_t n, int64_t k, oz_modset_t set, uint32_t route)
{
    Route rt;
    if (!valid_set(set) || !decode_route_for_set(set, route, &rt) || m < 0 || n < 0 || k < 0) return 0;
    if (resolve_schedule(set, k, n, true, &rt) != OZ_OK) return 0;
    return make_layout(m > 0 ? m : 1, n > 0 ? n : 1, k > 0 ? k : 1, set, rt).total;
}

oz_status_t oz_set_workspace(void *workspace, size_t bytes)
{
    int dev = 0;
    OZ_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return OZ_ERR_CUDA;
    if (workspace && (reinterpret_cast<uintptr_t>(workspace) & 255u)) return OZ_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_mutex);
    g_workspace[dev] = workspace;
    g_workspace_bytes[dev] = workspace ? bytes : 0;
    return OZ_OK;
}

oz_status_t oz_dgemm_ex(int64_t m, int64_t n, int64_t k, double alpha, const double *A, int64_t lda,
                        const double *B, int64_t ldb, double beta, double *C, int64_t ldc,
                        oz_modset_t set, uint32_t route, void *stream)
{
    int dev = 0;
    OZ_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return OZ_ERR_CUDA;
    char *ws = nullptr;
    size_t ws_bytes = 0;
    registered_workspace(dev, &ws, &ws_bytes);
    return dgemm_impl(m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, set, route,
                      static_cast<cudaStream_t>(stream), ws, ws_bytes);
}

oz_status_t oz_dgemm(int64_t m, int64_t n, int64_t k, const double *A, int64_t lda, const double *B,
                     int64_t ldb, double *C, int64_t ldc, oz_modset_t set, uint32_t route,
                     void *stream)
{
    return oz_dgemm_ex(m, n, k, 1.0, A, lda, B, ldb, 0.0, C, ldc, set, route, stream);
}

oz_status_t oz_dgemm_host(int64_t m, int64_t n, int64_t k, double alpha, const double *A_host,
                          int64_t lda, const double *B_host, int64_t ldb, double beta,
                          double *C_host, int64_t ldc, oz_modset_t set, uint32_t route,
                          void *stream)
{
    int dev = 0;
    OZ_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return OZ_ERR_CUDA;
    Route rt;
    if (!valid_set(set) || !decode_route_for_set(set, route, &rt)) return OZ_ERR_INVALID_ARG;
    if (m < 0 || n < 0 || k < 0) return OZ_ERR_INVALID_ARG;
    if (k > OZ_K_MAX || resolve_schedule(set, k, n, true, &rt) != OZ_OK) return OZ_ERR_UNSUPPORTED;
    if (m == 0 || n == 0) return OZ_OK;
    if (!C_host || ldc < m || (k > 0 && (!A_host || !B_host || lda < m || ldb < k)))
        return OZ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char *ws = nullptr;
    size_t ws_have = 0;
    registered_workspace(dev, &ws, &ws_have);
    int64_t kk = k > 0 ? k : 1;
    size_t core = make_layout(m, n, kk, set, rt).total;
    size_t bytesA = 8 * static_cast<size_t>(m) * kk, bytesB = 8 * static_cast<size_t>(kk) * n;
    size_t bytesC = 8 * static_cast<size_t>(m) * n;
    size_t offA = core, offB = offA + round_up(bytesA, 256), offC = offB + round_up(bytesB, 256);
    if (!ws || ws_have < offC + bytesC) return OZ_ERR_WORKSPACE;
    double *dA = reinterpret_cast<double *>(ws + offA);
    double *dB = reinterpret_cast<double *>(ws + offB);
    double *dC = reinterpret_cast<double *>(ws + offC);
    // Large outputs: C travels in column panels on two side streams, so that its upload overlaps
    // the deconstruction and the residue GEMMs, and the download of a finished panel overlaps the
    // upload and the reconstruction of the next ones (PCIe is full duplex).  The caller's stream
    // waits for both side streams before the call's work counts as done on it.
    int np = static_cast<int>(bytesC >> 26);                 // panels of at least 64 MiB
    if (np > kMaxPanels) np = kMaxPanels;
    if (np > n) np = static_cast<int>(n);
    if (k > 0 && np >= 2) {
        HostPipe *hp = nullptr;
        oz_status_t pst = ensure_pipe(dev, &hp);
        if (pst != OZ_OK) return pst;
        PanelPlan plan{};
        plan.np = np;
        for (int p = 0; p <= np; ++p) plan.col0[p] = n * p / np;
        plan.wait_before = beta != 0.0;
        plan.before = hp->c;
        plan.after = hp->r;
        OZ_CUDA_CHECK(cudaEventRecord(hp->start, s));          // the workspace may still be in use on s
        OZ_CUDA_CHECK(cudaStreamWaitEvent(hp->in, hp->start, 0));
        OZ_CUDA_CHECK(cudaStreamWaitEvent(hp->out, hp->start, 0));
        OZ_CUDA_CHECK(cudaMemcpy2DAsync(dA, 8 * m, A_host, 8 * lda, 8 * m, k, cudaMemcpyHostToDevice, hp->in));
        OZ_CUDA_CHECK(cudaMemcpy2DAsync(dB, 8 * k, B_host, 8 * ldb, 8 * k, n, cudaMemcpyHostToDevice, hp->in));
        OZ_CUDA_CHECK(cudaEventRecord(hp->ab, hp->in));
        if (beta != 0.0)
            for (int p = 0; p < np; ++p) {
                const int64_t j0 = plan.col0[p], cols = plan.col0[p + 1] - j0;
                OZ_CUDA_CHECK(cudaMemcpy2DAsync(dC + j0 * m, 8 * m, C_host + j0 * ldc, 8 * ldc, 8 * m, cols,
                                                cudaMemcpyHostToDevice, hp->in));
                OZ_CUDA_CHECK(cudaEventRecord(hp->c[p], hp->in));
            }
        OZ_CUDA_CHECK(cudaStreamWaitEvent(s, hp->ab, 0));
        oz_status_t st = dgemm_impl(m, n, k, alpha, dA, m, dB, kk, beta, dC, m, set, route, s, ws, core, &plan);
        if (st != OZ_OK) return st;
        for (int p = 0; p < np; ++p) {
            const int64_t j0 = plan.col0[p], cols = plan.col0[p + 1] - j0;
            OZ_CUDA_CHECK(cudaStreamWaitEvent(hp->out, hp->r[p], 0));
            OZ_CUDA_CHECK(cudaMemcpy2DAsync(C_host + j0 * ldc, 8 * ldc, dC + j0 * m, 8 * m, 8 * m, cols,
                                            cudaMemcpyDeviceToHost, hp->out));
        }
        OZ_CUDA_CHECK(cudaEventRecord(hp->done, hp->out));
        OZ_CUDA_CHECK(cudaStreamWaitEvent(s, hp->done, 0));
        return OZ_OK;
    }
    if (k > 0) {
        OZ_CUDA_CHECK(cudaMemcpy2DAsync(dA, 8 * m, A_host, 8 * lda, 8 * m, k, cudaMemcpyHostToDevice, s));
        OZ_CUDA_CHECK(cudaMemcpy2DAsync(dB, 8 * k, B_host, 8 * ldb, 8 * k, n, cudaMemcpyHostToDevice, s));
    }
    if (beta != 0.0)
        OZ_CUDA_CHECK(cudaMemcpy2DAsync(dC, 8 * m, C_host, 8 * ldc, 8 * m, n, cudaMemcpyHostToDevice, s));
    oz_status_t st = dgemm_impl(m, n, k, alpha, dA, m, dB, kk, beta, dC, m, set, route, s, ws, core);
    if (st != OZ_OK) return st;
    OZ_CUDA_CHECK(cudaMemcpy2DAsync(C_host, 8 * ldc, dC, 8 * m, 8 * m, n, cudaMemcpyDeviceToHost, s));
    return OZ_OK;
}

size_t oz_operand_bytes(int side, int64_t lines, int64_t k, oz_modset_t set, uint32_t route)
{
    Route rt;
    if (!valid_set(set) || !decode_route_for_set(set, route, &rt) || (side != 0 && side != 1) || lines < 0 ||
        k < 0 || k > OZ_K_MAX)
        return 0;
    if (resolve_schedule(set, k, 0, true, &rt) != OZ_OK) return 0;
    return operand_layout(side, lines > 0 ? lines : 1, k > 0 ? k : 1, set, rt).total;
}

size_t oz_product_workspace_bytes(int64_t m, int64_t n, oz_modset_t set)
{
    if (!valid_set(set) || m < 0 || n < 0) return 0;
    return residue_bytes_total(m > 0 ? m : 1, n > 0 ? n : 1, set);
}

oz_status_t oz_prepare_operand(int side, int64_t lines, int64_t k, const double *X, int64_t ldx,
                               oz_modset_t set, uint32_t route, void *operand, size_t bytes,
                               void *stream)
{
    Route rt;
    if (!valid_set(set) || !decode_route_for_set(set, route, &rt) || (side != 0 && side != 1))
        return OZ_ERR_INVALID_ARG;
    if (lines < 0 || k < 0) return OZ_ERR_INVALID_ARG;
    if (k > OZ_K_MAX) return OZ_ERR_UNSUPPORTED;
    if (resolve_schedule(set, k, 0, true, &rt) != OZ_OK) return OZ_ERR_UNSUPPORTED;
    if (rt.rule == 2) return OZ_ERR_UNSUPPORTED;      // the accurate rule derives the shifts from both operands
    if (lines == 0 || k == 0) return OZ_OK;           // nothing to keep: a product with k = 0 reads no operand
    if (!X || !operand || (reinterpret_cast<uintptr_t>(operand) & 255u) || (reinterpret_cast<uintptr_t>(X) & 7u) ||
        ldx < (side == 0 ? lines : k))
        return OZ_ERR_INVALID_ARG;
    const OperandLayout o = operand_layout(side, lines, k, set, rt);
    if (bytes < o.total) return OZ_ERR_WORKSPACE;
    oz_status_t st = ensure_device_ready();
    if (st != OZ_OK) return st;
    const OperandView v = operand_view(static_cast<char *>(operand), o);
    return launch_deconstruct(side, lines, k, X, ldx, set, rt, v.planes, v.stride, v.pitch, v.shift, v.scratch,
                              static_cast<cudaStream_t>(stream));
}

oz_status_t oz_dgemm_prepared(int64_t m, int64_t n, int64_t k, double alpha, const void *operandA,
                              const void *operandB, double beta, double *C, int64_t ldc,
                              oz_modset_t set, uint32_t route, void *stream)
{
    int dev = 0;
    OZ_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return OZ_ERR_CUDA;
    Route rt;
    bool trivial = true;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    oz_status_t st = check_product_args(m, n, k, alpha, beta, C, ldc, set, route, s, &rt, &trivial);
    if (st != OZ_OK || trivial) return st;
    if (rt.rule == 2) return OZ_ERR_UNSUPPORTED;      // prepared operands carry per-operand shifts
    if (rt.fallback || rt.fused) return OZ_ERR_UNSUPPORTED;   // both need the FP64 operands
    if (!operandA || !operandB || (reinterpret_cast<uintptr_t>(operandA) & 255u) ||
        (reinterpret_cast<uintptr_t>(operandB) & 255u))
        return OZ_ERR_INVALID_ARG;
    char *ws = nullptr;
    size_t ws_bytes = 0;
    registered_workspace(dev, &ws, &ws_bytes);
    if (!ws || ws_bytes < residue_bytes_total(m, n, set)) return OZ_ERR_WORKSPACE;
    st = ensure_device_ready();
    if (st != OZ_OK) return st;
    const OperandView a = operand_view(static_cast<char *>(const_cast<void *>(operandA)), operand_layout(0, m, k, set, rt));
    const OperandView b = operand_view(static_cast<char *>(const_cast<void *>(operandB)), operand_layout(1, n, k, set, rt));
    if (g_stage_events_on[dev]) {
        // no deconstruction in this call: the first three events coincide
        OZ_CUDA_CHECK(cudaEventRecord(g_stage_events[dev][0], s));
        OZ_CUDA_CHECK(cudaEventRecord(g_stage_events[dev][1], s));
    }
    return product_impl(m, n, k, alpha, a, b, beta, C, ldc, set, rt, s, ws, dev, nullptr);
}

oz_status_t oz_deconstruct(int side, int64_t lines, int64_t k, const double *X, int64_t ldx,
                           oz_modset_t set, uint32_t route, uint8_t *planes, int64_t plane_stride,
                           int64_t row_pitch, int32_t *shift, void *scratch, void *stream)
{
    Route rt;
    if (!valid_set(set) || !decode_route_for_set(set, route, &rt) || (side != 0 && side != 1))
        return OZ_ERR_INVALID_ARG;
    if (lines < 0 || k < 0) return OZ_ERR_INVALID_ARG;
    if (k > OZ_K_MAX) return OZ_ERR_UNSUPPORTED;
    if (resolve_schedule(set, k, 0, false, &rt) != OZ_OK) return OZ_ERR_UNSUPPORTED;
    if (lines == 0) return OZ_OK;
    if (!planes || !shift || !scratch || (k > 0 && !X)) return OZ_ERR_INVALID_ARG;
    if (row_pitch < k || row_pitch < 16 || (row_pitch & 15) || (plane_stride & 15) ||
        plane_stride < lines * row_pitch || (reinterpret_cast<uintptr_t>(planes) & 15u) ||
        (reinterpret_cast<uintptr_t>(scratch) & 255u) || (reinterpret_cast<uintptr_t>(shift) & 3u) ||
        (reinterpret_cast<uintptr_t>(X) & 7u))
        return OZ_ERR_INVALID_ARG;
    if (k > 0 && ldx < (side == 0 ? lines : k)) return OZ_ERR_INVALID_ARG;
    oz_status_t st = ensure_device_ready();
    if (st != OZ_OK) return st;
    return launch_deconstruct(side, lines, k, X, ldx, set, rt, planes, plane_stride, row_pitch, shift,
                              scratch, static_cast<cudaStream_t>(stream));
}

oz_status_t oz_residue_gemm(int64_t m, int64_t n, int64_t k, const uint8_t *PA, int64_t strideA,
                            int64_t pitchA, const uint8_t *PB, int64_t strideB, int64_t pitchB,
                            oz_modset_t set, uint32_t route, void *R, int64_t ldr,
                            int64_t mod_stride, void *stream)
{
    Route rt;
    if (!valid_set(set) || !decode_route_for_set(set, route, &rt)) return OZ_ERR_INVALID_ARG;
    if (m < 0 || n < 0 || k < 0) return OZ_ERR_INVALID_ARG;
    if (k > OZ_K_MAX) return OZ_ERR_UNSUPPORTED;
    if (resolve_schedule(set, k, 0, false, &rt) != OZ_OK) return OZ_ERR_UNSUPPORTED;
    if (m == 0 || n == 0) return OZ_OK;
    if (!PA || !PB || !R || ldr < m || mod_stride < n * ldr) return OZ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(R) % static_cast<uintptr_t>(residue_bytes(set))) return OZ_ERR_INVALID_ARG;
    if ((pitchA & 15) || (pitchB & 15) || (strideA & 15) || (strideB & 15) || pitchA < k ||
        pitchB < k || pitchA < 16 || pitchB < 16 || strideA < m * pitchA || strideB < n * pitchB ||
        (reinterpret_cast<uintptr_t>(PA) & 15u) || (reinterpret_cast<uintptr_t>(PB) & 15u))
        return OZ_ERR_INVALID_ARG;
    oz_status_t st = ensure_device_ready();
    if (st != OZ_OK) return st;
    return launch_residue_gemm(m, n, k, PA, strideA, pitchA, PB, strideB, pitchB, set, rt, R, ldr,
                               mod_stride, false, false, static_cast<cudaStream_t>(stream));
}

oz_status_t oz_reconstruct(int64_t m, int64_t n, const void *R, int64_t ldr, int64_t mod_stride,
                           const int32_t *shiftA, const int32_t *shiftB, oz_modset_t set,
                           double alpha, double beta, double *C, int64_t ldc, void *stream)
{
    if (!valid_set(set) || m < 0 || n < 0) return OZ_ERR_INVALID_ARG;
    if (!(alpha == 1.0 || alpha == -1.0) || !(beta == 0.0 || beta == 1.0)) return OZ_ERR_UNSUPPORTED;
    if (m == 0 || n == 0) return OZ_OK;
    if (!R || !shiftA || !shiftB || !C || ldr < m || mod_stride < n * ldr || ldc < m)
        return OZ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(R) % static_cast<uintptr_t>(residue_bytes(set)) ||
        (reinterpret_cast<uintptr_t>(shiftA) & 3u) || (reinterpret_cast<uintptr_t>(shiftB) & 3u) ||
        (reinterpret_cast<uintptr_t>(C) & 7u))
        return OZ_ERR_INVALID_ARG;
    oz_status_t st = ensure_device_ready();
    if (st != OZ_OK) return st;
    return launch_reconstruct(m, n, R, ldr, mod_stride, shiftA, shiftB, set, alpha, beta, C, ldc,
                              static_cast<cudaStream_t>(stream));
}

oz_status_t oz_query_status(void *stream)
{
    oz_status_t st = ensure_device_ready();
    if (st != OZ_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned int word[4] = {0, 0, 0, 0};
    OZ_CUDA_CHECK(cudaStreamSynchronize(s));
    OZ_CUDA_CHECK(cudaMemcpyFromSymbol(word, g_status, sizeof(word)));
    OZ_CUDA_CHECK(cudaMemcpyToSymbol(g_status, kStatusReset, sizeof(word)));   // word 4 has its own query
    if (cudaGetLastError() != cudaSuccess) return OZ_ERR_CUDA;
    if (word[0] & (1u << OZ_ERR_TIMEOUT)) return OZ_ERR_TIMEOUT;
    if (word[0] & (1u << OZ_ERR_NONFINITE_INPUT)) return OZ_ERR_NONFINITE_INPUT;
    // exponent-span check: an operand that was not scanned since the last query counts as flat
    const uint64_t qa = word[1] > 65536u ? 65536u : word[1], qb = word[2] > 65536u ? 65536u : word[2];
    if (word[3] != 0u && qa * qb < static_cast<uint64_t>(word[3])) return OZ_ERR_RANGE;
    return OZ_OK;
}

oz_status_t oz_query_fallback_rows(void *stream, int64_t *rows)
{
    if (!rows) return OZ_ERR_INVALID_ARG;
    oz_status_t st = ensure_device_ready();
    if (st != OZ_OK) return st;
    OZ_CUDA_CHECK(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    unsigned int count = 0;
    const unsigned int zero = 0;
    OZ_CUDA_CHECK(cudaMemcpyFromSymbol(&count, g_status, sizeof(count), 4 * sizeof(unsigned int)));
    OZ_CUDA_CHECK(cudaMemcpyToSymbol(g_status, &zero, sizeof(zero), 4 * sizeof(unsigned int)));
    *rows = static_cast<int64_t>(count);
    return OZ_OK;
}

oz_status_t oz_set_stage_events(void *const *events)
{
    int dev = 0;
    OZ_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return OZ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    g_stage_events_on[dev] = false;
    if (events)
        for (int i = 0; i < 5; ++i)
            if (!events[i]) return OZ_ERR_INVALID_ARG;
    for (int i = 0; i < 5; ++i)
        g_stage_events[dev][i] = events ? static_cast<cudaEvent_t>(events[i]) : nullptr;
    g_stage_events_on[dev] = events != nullptr;
    return OZ_OK;
}

uint64_t oz_launch_count(void) { return g_launches.load(); }

const char *oz_status_string(oz_status_t status)
{
    switch (status) {
        case OZ_OK: return "ok";
        case OZ_ERR_INVALID_ARG: return "invalid argument";
        case OZ_ERR_UNSUPPORTED: return "unsupported (k above OZ_K_MAX, or alpha/beta not in {+-1}/{0,1})";
        case OZ_ERR_WORKSPACE: return "workspace missing or too small";
        case OZ_ERR_CUDA: return "CUDA call failed";
        case OZ_ERR_NONFINITE_INPUT: return "Inf/NaN in an operand";
        case OZ_ERR_RANGE: return "exponent-span check: operands too unevenly scaled for FP64-grade accuracy with this modulus set";
        case OZ_ERR_TIMEOUT: return "bounded device wait ran out";
    }
    return "unknown status";
}

}  // extern "C"
