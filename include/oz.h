/*
 * oz.h -- C ABI of the B200 (sm_100a) Ozaki Scheme II emulated-FP64 GEMM library.
 *
 * The library computes C = A B for FP64 matrices through exact integer residue
 * arithmetic on the FP8 / INT8 tensor cores (paper Sec. 2, "The scheme in
 * equations", Eq. 1-5, and "The FP8 variant", Eq. 6-7):
 *   1. deconstruction (Algorithm 2): per-row / per-column power-of-two scaling, quantisation
 *      to integers, centred residues modulo each modulus of the set, two-limb digit
 *      split with the carry of Lemma 1, stored as K-major 8-bit planes;
 *   2. residue products (Algorithm 1, the loop over moduli): three exact plane GEMMs per modulus,
 *      combined and reduced modulo m_i in the epilogue (Eq. 8 for non-squares,
 *      weights {1,s,s} for squares m = s^2);
 *   3. reconstruction (Algorithm 3, Eq. 4-5): CRT, lift to [-M/2, M/2), inverse scaling,
 *      one rounding to FP64.
 *
 * General conventions
 *   - Matrices are column-major, no transposes: A is m x k (lda >= m), B is k x n
 *     (ldb >= k), C is m x n (ldc >= m).
 *   - Every pointer is a DEVICE pointer owned by the caller unless a comment says
 *     "host", aligned to its element type (8 bytes for matrices, 4 for shifts; OZ_ERR_INVALID_ARG
 *     otherwise).  The library never allocates or frees device memory; scratch comes
 *     from the workspace registered with oz_set_workspace().
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is the
 *     default stream), or on internal streams that fork from it and join it again inside the
 *     call, so that ordering on `stream` is all a caller needs.  No call synchronises the host
 *     except oz_query_status().  The whole-method entry points (oz_dgemm, oz_dgemm_ex,
 *     oz_dgemm_host) create their internal stream and events on a device's first such call:
 *     make that call outside a stream capture.  The stage entry points use `stream` only.
 *   - Host-detectable errors return at once with nothing enqueued.  Conditions
 *     found on the device (non-finite input, a bounded wait that ran out) set a
 *     sticky per-device status word that oz_query_status() returns and clears.
 *     Kernels never trap and never spin without a limit.
 *   - m, n or k equal to zero is OZ_OK (k = 0 gives C = 0, or C unchanged for beta = 1).
 *   - Non-finite contract: an Inf or NaN anywhere in row i of A (column j of B)
 *     makes every C(i,:) (C(:,j)) NaN and sets OZ_ERR_NONFINITE_INPUT.
 *   - Range of the result: the product is rounded once to 53 bits and then scaled by a power of
 *     two.  Where that scaling lands below the normal range (|C_ij| < 2^-1022) the value is rounded a
 *     second time, to the subnormal grid, and where it lands above the largest finite number it
 *     becomes infinite; such outputs are outside the single-rounding contract.
 *   - One FP32 accumulator of the FP8 route stays exact to k = 32768 (Lemma 1 and the accumulation
 *     invariant of Algorithm 2), an INT32 one to 131071 (native residues) or 4 million (digits).
 *     A longer k is split inside the residue-GEMM kernel into K segments with an accumulator each,
 *     reduced modulo m_i and added in the residue domain; the shifts are those of the whole k.
 *     k is limited to OZ_K_MAX.
 */
#ifndef OZ_H_
#define OZ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    OZ_OK = 0,
    OZ_ERR_INVALID_ARG = 1,     /* null pointer, negative size, bad leading dimension, bad enum */
    OZ_ERR_UNSUPPORTED = 2,     /* k > OZ_K_MAX, alpha/beta outside {+-1}/{0,1}, OZ_SCALE_ACCURATE
                                 * through a per-operand entry point or with k > 16384             */
    OZ_ERR_WORKSPACE = 3,       /* no workspace registered, or it is too small                  */
    OZ_ERR_CUDA = 4,            /* a CUDA runtime / driver call failed                          */
    OZ_ERR_NONFINITE_INPUT = 5, /* device: Inf/NaN met in an operand                            */
    OZ_ERR_RANGE = 6,           /* device: the exponent-span check flags the operands (see below); the
                                 * results are computed all the same                             */
    OZ_ERR_TIMEOUT = 7          /* device: a bounded barrier wait ran out                       */
} oz_status_t;

/* Modulus sets: S = the published 12-modulus set (Sec. 2, step (ii));
 * E = the hybrid set, six squares of S plus seven byte moduli ("Candidate E");
 * A = the all-byte set of fifteen moduli, 117.8 bits ("Candidate A"). */
typedef enum { OZ_SET_S = 0, OZ_SET_E = 1, OZ_SET_A = 2 } oz_modset_t;

/* route bit field: one substrate, one quantiser, one scale rule (0 picks the default) */
#define OZ_SUB_FP8      0x001u  /* planes are E4M3 bytes, FP32 accumulation (default)          */
#define OZ_SUB_INT8     0x002u  /* same digits as two's-complement bytes, INT32 accumulation   */
#define OZ_SUB_INT8_NATIVE 0x004u /* set A only: the centred residue of a byte modulus IS the INT8
                                   * operand -- one plane and one product per modulus (Sec. 2, "The
                                   * substrate transition": alpha_INT8 = r + 1 = 16 passes)            */
#define OZ_QUANT_RN     0x010u  /* round to nearest, ties to even (variant Ozaki-II-RN, default) */
#define OZ_QUANT_TZ     0x020u  /* truncate toward zero (variant Ozaki-II-TZ)                  */
#define OZ_SCALE_MAXEXP 0x100u  /* shift from the largest exponent of the line (Eq. 2 read literally) */
#define OZ_SCALE_CS     0x200u  /* shift from the 2-norm of the line, Cauchy-Schwarz bound (default) */
#define OZ_SCALE_ACCURATE 0x400u /* accurate mode (Sec. 2 "The FP8 variant": one additional FP8 GEMM
                                  * estimates an input magnitude bound, the "+1" of the 3r + 1 passes):
                                  * every element gives an E4M3-exact magnitude digit >= |x| 2^(4-E) (E the
                                  * largest exponent of its line), one extra tensor-core product of the two
                                  * digit planes bounds (|A||B|)_ij, and the shifts come from the row and
                                  * column maxima of that product, so that every |c'_ij| stays inside the
                                  * CRT range.  Whole-method calls only (the shifts of one operand depend on
                                  * the other): oz_dgemm, oz_dgemm_ex, oz_dgemm_host; k <= 16384.            */

/* Accumulator schedule of the residue GEMMs for non-square moduli on the two digit substrates.
 * MERGED: two accumulators per modulus, d e = -15 [d0 e0 + (-16 d1) e1] + 16 (d0+d1)(e0+e1)
 * (discussion of Table "tuples", N_acc = 2).  The plane counts stay those of the table.
 *   FP8:  the A operand stores the pre-scaled -16*d1 in the place of d1 (plane order d0, -16*d1,
 *         d0+d1; d1 enters only through d1 e1), B is unchanged.  One merged accumulator is exact
 *         while it stays below 2^24: k <= 4097 for set S, k <= 15420 for sets E and A.
 *   INT8: -16*d1 does not fit a byte, so the factor is shared: A stores -d0, 4*d1, d0+d1 and B stores
 *         e0, 4*e1, e0+e1; the accumulator (-d0) e0 + (4 d1)(4 e1) is the negative of the bracket and
 *         takes the weight +15.  Its term is at most 4292, exact in INT32 for k <= 500 000.
 * A longer k is cut into equal K segments no longer than that, each with an accumulator of its own
 * that is reduced modulo m_i before the segments are added (split-K inside the kernel; the residues
 * are the same).
 * SEPARATE: the three accumulators of Eq. 8.  With neither bit, oz_dgemm / oz_dgemm_ex /
 * oz_dgemm_host pick MERGED on the digit substrates (their planes are internal), and the stage entry
 * points use SEPARATE.  Planes written with MERGED must be multiplied with MERGED.  Not defined for
 * OZ_SUB_INT8_NATIVE (one plane per modulus). */
#define OZ_ACC_MERGED   0x1000u
#define OZ_ACC_SEPARATE 0x2000u

/* Reconstruction of the whole-method calls with the CRT recombination hosted on the INT8 tensor pipe
 * (Algorithm 3, the "[INT8-TENSOR + SIMT]" branch: about r multiply-accumulates per output as one
 * small unsigned 8-bit product, then carry, lift and the single rounding in integer arithmetic).
 * Same results bit for bit.  The default form evaluates the same weighted sum in exact FP64 chunks;
 * on B200, whose FP64 pipe is as wide as its integer pipe, that form is about 1.8 times faster, so
 * this bit is for comparison and for parts with a narrow FP64 pipe.  Ignored by the stage entry points. */
#define OZ_RECON_TENSOR 0x4000u

/* Out-of-range rows on the native FP64 path (Algorithm 1, last line: "ESC check; native-FP64 fallback
 * for out-of-range rows"; Algorithm 3: "ESC range check; re-issue out-of-range rows on the native-FP64
 * path").  The paper names the step; criterion and arithmetic are the library's reading.  With this bit
 * oz_dgemm / oz_dgemm_ex apply the exponent-span check of oz_query_status() row by row: row i of the
 * product is out of range when  min(q(a_i), 2^16) * min(min_j q(b_j), 2^16) < threshold  (q = floor(2^16
 * phi^2), same threshold).  Such rows are left out of the reconstruction and computed in FP64 from the
 * caller's old C: each entry is the compensated inner product of its row of A and column of B taken in
 * the order kk = 0 .. k-1 (product error by one fused multiply-add, addition error by the error-free
 * sum of two doubles, both collected in a second double that is added at the end), then
 * C = alpha P or C + alpha P.  The value depends on the data alone, and it meets 2u (|A||B|)_ij like the
 * emulated rows.  Cost: about ten FP64 operations per multiply-add on the SIMT FP64 pipe, so a call in
 * which every row fails runs far below the emulated rate -- as the paper says, the fallback does not
 * accelerate.  OZ_ERR_RANGE is still reported (informational).  oz_query_fallback_rows() returns how
 * many rows were re-issued.  Needs OZ_SCALE_CS (the check is defined on its scan); not combined with
 * OZ_RECON_TENSOR; OZ_ERR_UNSUPPORTED from oz_dgemm_host and oz_dgemm_prepared; ignored by the stage
 * entry points.  Workspace: oz_workspace_bytes() with the same route (5 m + 768 bytes more). */
#define OZ_FALLBACK_FP64 0x8000u

/* Storage mode F for tall-skinny products (Sec. "Storage Modes", mode F; "O4: pipelining"): the planes
 * of A are never written to memory.  oz_dgemm / oz_dgemm_ex then run only the scan of A (its shifts),
 * and the product kernel converts each 64-row tile of A into plane bytes inside the shared-memory ring
 * that feeds the tensor core, four moduli per pass over the tile (the paper's modulus blocking with
 * n_blk = 4: A is read and quantised r/4 times).  B is deconstructed as always.  Same residues, same
 * result, bit for bit.  Applies when n <= 128, the substrate is FP8 or INT8 digits (merged schedule,
 * which the bit implies), and k is within the exact depth of one accumulator (k <= 4097 on set S,
 * 15420 on sets E and A for FP8; 262144 for INT8 digits); OZ_ERR_UNSUPPORTED otherwise, and with
 * OZ_SCALE_ACCURATE, OZ_RECON_TENSOR, OZ_FALLBACK_FP64, oz_dgemm_host and oz_dgemm_prepared.  Ignored by
 * the stage entry points. */
#define OZ_STORAGE_FUSED 0x10000u

#define OZ_K_MAX 1048576
#define OZ_NONFINITE_SHIFT INT32_MIN  /* value of shift[] for a line that holds Inf/NaN */

/* Number of moduli r and of stored planes p_store of a set (Table "tuples": 12/30, 13/33).
 * Returns OZ_ERR_INVALID_ARG for an unknown set.  `moduli` (host, may be NULL) receives r ints. */
oz_status_t oz_set_info(oz_modset_t set, int *r, int *p_store, int *moduli);

/* Stored planes of a set on the substrate named by `route`: 30 / 33 / 44 for S / E / A with
 * two-limb digits, 15 for set A with OZ_SUB_INT8_NATIVE; 0 for an invalid combination. */
int oz_plane_count(oz_modset_t set, uint32_t route);

/* Same, for the operand on `side` (0: A, 1: B).  The counts of the two sides are equal on every
 * route (with OZ_ACC_MERGED the re-scaled planes take the places of the plain ones); the function remains
 * for callers that size the two plane arrays separately. */
int oz_plane_count_side(oz_modset_t set, uint32_t route, int side);

/* Bytes of one stored residue: 2 (uint16) for sets S and E, 1 (uint8) for the all-byte set A, whose
 * moduli do not exceed 256; 0 for an unknown set.  This is the element type of the array R of
 * oz_residue_gemm and oz_reconstruct. */
size_t oz_residue_elem_bytes(oz_modset_t set);

/* Pitch in bytes of one plane row for inner dimension k: k rounded up to 16 (TMA stride rule). */
int64_t oz_row_pitch(int64_t k);

/* Bytes of scratch that oz_dgemm needs for this shape (planes of A and B, residues, shifts). */
size_t oz_workspace_bytes(int64_t m, int64_t n, int64_t k, oz_modset_t set, uint32_t route);

/* Register caller-owned device scratch (256-byte aligned) for oz_dgemm / oz_dgemm_ex on the
 * current device.  The library keeps only the pointer; the caller frees it after the last call
 * has finished.  Passing NULL unregisters. */
oz_status_t oz_set_workspace(void *workspace, size_t bytes);

/* C = A B  (Sec. 2: the whole method).  Needs a registered workspace of at least
 * oz_workspace_bytes().  Kernels launched: scan, deconstruct (A and B), residue GEMM, reconstruct. */
oz_status_t oz_dgemm(int64_t m, int64_t n, int64_t k, const double *A, int64_t lda,
                     const double *B, int64_t ldb, double *C, int64_t ldc, oz_modset_t set,
                     uint32_t route, void *stream);

/* C = beta C + alpha A B with alpha in {+1,-1}, beta in {0,1} (the HPL trailing update
 * C <- C - A B of Sec. "HPL" is alpha = -1, beta = 1).  With beta = 1 the result carries two
 * roundings: the method's single rounding of the product, then the FP64 addition. */
oz_status_t oz_dgemm_ex(int64_t m, int64_t n, int64_t k, double alpha, const double *A,
                        int64_t lda, const double *B, int64_t ldb, double beta, double *C,
                        int64_t ldc, oz_modset_t set, uint32_t route, void *stream);

/* Same as oz_dgemm_ex but A, B, C are HOST pointers (pinned memory recommended: copies from
 * pageable memory do not overlap anything).  The operands are copied to staging areas inside the
 * registered workspace, which must hold oz_workspace_bytes() + 8 (m k + k n + m n) bytes, and C is
 * copied back; the call returns after enqueueing (the host buffers must stay valid until the stream
 * has drained).  When C is 128 MiB or more it travels in up to 16 column panels on two internal
 * streams: its upload overlaps the deconstruction and the residue GEMMs, and each panel is downloaded
 * while later ones are still uploaded and reconstructed.  `stream` waits for those internal streams,
 * so work enqueued on it afterwards, or a synchronisation of it, sees the finished C.  The internal
 * streams and events are created on a device's first such call (not inside a stream capture). */
oz_status_t oz_dgemm_host(int64_t m, int64_t n, int64_t k, double alpha, const double *A_host,
                          int64_t lda, const double *B_host, int64_t ldb, double beta,
                          double *C_host, int64_t ldc, oz_modset_t set, uint32_t route,
                          void *stream);

/* Planes kept across calls (storage mode P of Sec. "Storage Modes"; paragraph "O1: convert-once
 * residue-plane workspace"): an operand that takes part in several products -- the panel of an HPL
 * trailing update, the operator of an iterative solver -- is deconstructed once into a caller-owned
 * block and then multiplied any number of times.
 *
 * oz_operand_bytes: size of that block for `lines` rows of A (side 0) or columns of B (side 1) and
 * inner dimension k; 0 for invalid arguments.  The block holds the shifts, the planes in the layout
 * and pitch that the whole-method calls use internally (not the layout of oz_deconstruct), and the
 * scan scratch; its content is opaque.
 * oz_prepare_operand: deconstructs X (same conventions as oz_deconstruct) into `operand` (device
 * memory, 256-byte aligned, at least oz_operand_bytes()).  Scaling rule, quantiser, substrate and set
 * come from `route` / `set` and must be the same in every call that uses the block.
 * oz_dgemm_prepared: C = beta C + alpha A B from two prepared operands (A: m lines, B: n lines, same k,
 * set and route).  Needs a registered workspace of oz_product_workspace_bytes(m, n, set) bytes (the
 * residues); launches the residue GEMMs and the reconstruction only.  The result is bit-identical to
 * oz_dgemm_ex on the same matrices: the shifts of a line depend on that line alone. */
size_t oz_operand_bytes(int side, int64_t lines, int64_t k, oz_modset_t set, uint32_t route);
size_t oz_product_workspace_bytes(int64_t m, int64_t n, oz_modset_t set);
oz_status_t oz_prepare_operand(int side, int64_t lines, int64_t k, const double *X, int64_t ldx,
                               oz_modset_t set, uint32_t route, void *operand, size_t bytes,
                               void *stream);
oz_status_t oz_dgemm_prepared(int64_t m, int64_t n, int64_t k, double alpha, const void *operandA,
                              const void *operandB, double beta, double *C, int64_t ldc,
                              oz_modset_t set, uint32_t route, void *stream);

/* Deconstruction of one operand (Algorithm 2; scaling of Eq. 1).
 *   side 0: X is m x k column-major, lines = m rows,    element (i,kk) at X[i + kk*ldx]
 *   side 1: X is k x n column-major, lines = n columns, element (kk,j) at X[kk + j*ldx]
 * Outputs: shift[lines] (int32; sigma_i or tau_j of Eq. 1, OZ_NONFINITE_SHIFT for a line with
 * Inf/NaN) and p_store planes, plane p / line l / inner index kk at
 *   planes[p*plane_stride + l*row_pitch + kk],
 * in the set's modulus order, plane order d0, d1[, d0+d1] per modulus; bytes kk in [k,row_pitch)
 * are written as zero.  row_pitch >= k and plane_stride >= lines*row_pitch, both multiples of 16;
 * `planes` 16-byte aligned.  `scratch` is 16*lines + 256 bytes of device memory (256-byte aligned). */
oz_status_t oz_deconstruct(int side, int64_t lines, int64_t k, const double *X, int64_t ldx,
                           oz_modset_t set, uint32_t route, uint8_t *planes,
                           int64_t plane_stride, int64_t row_pitch, int32_t *shift,
                           void *scratch, void *stream);

/* oz_deconstruct for callers that cannot allocate device memory (no counterpart in the paper: it
 * is a packaging variant, not a step of the method).  Identical to oz_deconstruct except that the
 * scan scratch is a fixed array inside the library (16 * OZ_STATIC_MAX_LINES + 256 bytes, held by
 * every GPU that loads the library until the process exits), so there is no `scratch` argument
 * and the call performs no device allocation of any kind.
 *   - lines > OZ_STATIC_MAX_LINES returns OZ_ERR_WORKSPACE with nothing enqueued.
 *   - The first call on a device looks the array's device address up (a host-side query, once per
 *     device, with that device current); make that first call before starting a stream capture.
 *   - All calls on a device share the one array.  Each call clears what it uses before use, so
 *     results never depend on an earlier call; but two calls whose kernels overlap on the GPU
 *     (different streams, no ordering between them) race on it.  Serialise them. */
#define OZ_STATIC_MAX_LINES 262144
oz_status_t oz_deconstruct_static(int side, int64_t lines, int64_t k, const double *X, int64_t ldx,
                                  oz_modset_t set, uint32_t route, uint8_t *planes,
                                  int64_t plane_stride, int64_t row_pitch, int32_t *shift,
                                  void *stream);

/* Residue products (Eq. 3 through the plane identities of Sec. 2 "FP8 variant" and Eq. 8):
 * for every modulus i,  R_i = (A_i B_i) mod m_i  from the stored planes of A (lines = m) and
 * B (lines = n), on the tensor cores.  Output R[i*mod_stride + j*ldr + row], the canonical residue
 * in [0, m_i) as an unsigned integer of oz_residue_elem_bytes(set) bytes (uint16 for S and E, uint8
 * for A; device memory).  ldr >= m, mod_stride >= n*ldr (in elements); rows whose byte offset is a
 * multiple of 16 (R 16-byte aligned, ldr and mod_stride multiples of 8 resp. 16 elements) take the
 * fast vector stores, anything else a slower element-wise path with the same result.  Planes as
 * written by oz_deconstruct with the same set and substrate; plane bases 16-byte aligned, pitches
 * and strides multiples of 16. */
oz_status_t oz_residue_gemm(int64_t m, int64_t n, int64_t k, const uint8_t *PA,
                            int64_t plane_strideA, int64_t row_pitchA, const uint8_t *PB,
                            int64_t plane_strideB, int64_t row_pitchB, oz_modset_t set,
                            uint32_t route, void *R, int64_t ldr, int64_t mod_stride,
                            void *stream);

/* Reconstruction (Algorithm 3; Eq. 4-5 and the final step of Sec. 2 (iv)): the integer
 * c'_ij in [-M/2, M/2) congruent to the residues, times 2^-(shiftA[i]+shiftB[j]), rounded once;
 * C = alpha P (beta = 0) or C = C + alpha P (beta = 1).  The CRT is evaluated exactly.  R has the
 * layout and element type that oz_residue_gemm writes for `set`; an entry may be any representative
 * of its residue class below 2 m_i that fits the element type, not only the canonical one (adding
 * m_i to c_i changes the CRT sum by a multiple of M). */
oz_status_t oz_reconstruct(int64_t m, int64_t n, const void *R, int64_t ldr,
                           int64_t mod_stride, const int32_t *shiftA, const int32_t *shiftB,
                           oz_modset_t set, double alpha, double beta, double *C, int64_t ldc,
                           void *stream);

/* Synchronises `stream`, then returns and clears the device status of the current device: the first
 * that applies of OZ_ERR_CUDA, OZ_ERR_TIMEOUT, OZ_ERR_NONFINITE_INPUT, OZ_ERR_RANGE, else OZ_OK.
 *
 * OZ_ERR_RANGE is the exponent-span check (Algorithm 1, last line: "ESC check"; the paper leaves the
 * criterion to its sources, this is the library's reading).  With the norm-based scale rule
 * (OZ_SCALE_CS, the default) the scan also measures how evenly every line spreads its magnitude,
 *     phi(x) = ||x||_1 / (sqrt(k) ||x||_2)   (1: constant line, 1/sqrt(k): one spike),
 * and the status reports OZ_ERR_RANGE when, for the operands deconstructed since the last query,
 *     min_i phi(a_i)^2 * min_j phi(b_j)^2  <  (16/3) 2^104 / ((M-1)/2),
 * i.e. when the rounding-error model predicts a typical error above an eighth of 2u (|A||B|)_ij: the
 * modulus set is then too small for FP64-grade accuracy on this data (escalate to a larger set, e.g.
 * OZ_SET_A, or use native FP64 for it).  Purely informational: every result is still computed and
 * matches the method's definition.  Not evaluated with OZ_SCALE_MAXEXP or OZ_SCALE_ACCURATE. */
oz_status_t oz_query_status(void *stream);

/* Synchronises `stream`, stores in *rows (host) the number of rows that calls with OZ_FALLBACK_FP64
 * re-issued on the native FP64 path on the current device since the last such query, and clears it. */
oz_status_t oz_query_fallback_rows(void *stream, int64_t *rows);

/* Optional per-stage timing hook for benchmarks (the paper's Algorithm 1 prices each stage
 * separately), kept per device: it applies to the device that is current when it is set.  `events`
 * is a HOST array of 5 cudaEvent_t handles (as void*), or NULL to switch the hook off.  While set,
 * oz_dgemm / oz_dgemm_ex / oz_dgemm_prepared record them on the call's stream: [0] before the
 * first kernel, [1] after the deconstruction of A, [2] once the deconstruction of B -- which runs
 * next to A's on an internal stream that forks from and joins the call's stream -- has finished
 * too, [3] after the residue GEMMs, [4] after the reconstruction.  The handles are copied; the
 * caller owns the events. */
oz_status_t oz_set_stage_events(void *const *events);

/* Number of kernels launched by the library on this process since load (for benchmarks). */
uint64_t oz_launch_count(void);

/* Human-readable name of a status code (host string, never NULL). */
const char *oz_status_string(oz_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* OZ_H_ */
