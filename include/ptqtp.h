/* ptqtp.h -- C ABI of the PTQTP dual-trit-plane decode linear layer for NVIDIA B200 (sm_100a).
 *
 * A weight matrix W [N out, K in] is stored as two ternary planes T1, T2 in {-1,0,+1}^{N x K} and
 * two scale tables alpha1, alpha2 with one fp16 value per output row per group of 128 input columns
 * (Eq. 1-2: W ~ diag(alpha1) T1 + diag(alpha2) T2; Sec. 2.3 "Batch Processing": the scales are
 * per group-row after reshaping n x d to (nd/G) x G with G = 128).  The layer computes
 *
 *     y[i] = sum_g ( alpha1[i,g] * sum_{j in g} T1[i,j] x[j]  +  alpha2[i,g] * sum_{j in g} T2[i,j] x[j] )
 *
 * where a trit contributes +x, -x or nothing (Sec. 4 "Hardware Efficiency") and the per-group
 * scale is the only multiplication.
 *
 * Conventions for every call
 *   - Pointers marked "device" are CUDA device pointers on the current device; "host" are host
 *     pointers.  The caller owns every buffer.  Except where an entry point says otherwise the
 *     library never allocates, frees or synchronises: calls enqueue work on `stream` (a
 *     cudaStream_t passed as void*, NULL = the default stream) and return after the launch.
 *   - Device buffers must be 16-byte aligned (PTQTP_ERR_ALIGN otherwise).
 *   - Host-detectable errors return a negative status and launch nothing.
 *   - Errors only the device can see (a plane entry outside {-1,0,1}, a bad header) are written
 *     to `*dev_status` (a device int32 the caller zeroes beforehand and reads after syncing); the
 *     kernel still completes normally.  `dev_status` may be NULL where noted.
 *   - K must be a positive multiple of 128 (the group reshape of Sec. 2.3 presumes it); N >= 1.
 *   - Matrices are row-major: T[i*K + j], alpha[i*(K/128) + g], X[m*K + j], Y[m*N + i].
 *   - fp16 values cross the ABI as their 16-bit patterns (uint16_t).
 *
 * Packed format "PTQTP-B200 v1" (chosen for 128-bit coalesced streaming; the storage model of
 * Appendix B "Memory Saving": 2 bits per trit per plane + one fp16 scale per plane per group):
 *   [0, 256)            header: magic "PTQTPB2\0", u32 version(1), u32 format(1), i32 N, i32 K,
 *                       i32 group(128), i32 K_pad, u64 codes_offset, u64 scales_offset, u64 total bytes
 *   codes  (at 256)     N * (K_pad/1024) chunks of 512 bytes, row-major in (row, slice).  K_pad = K
 *                       rounded up to a multiple of 1024; padding columns hold trit 0.
 *                       Chunk (i, s) covers columns s*1024 .. s*1024+1023 of row i as 32 lane blocks
 *                       of 16 bytes; lane block l covers the 32 columns s*1024 + 32*l + e, e = 0..31,
 *                       as four little-endian u32 words:
 *                         word 0: plane 1, e = 0..15      word 1: plane 1, e = 16..31
 *                         word 2: plane 2, e = 0..15      word 3: plane 2, e = 16..31
 *                       In a word, column offset e' = e mod 16 sits in the 16-bit half h = e'/8 at bits
 *                       [16h + 2(e' mod 8), +1] as the code q = trit + 1 in {0,1,2} (3 never occurs).
 *   scales (after codes) N * (K_pad/128) pairs (alpha1 fp16, alpha2 fp16), row-major; pairs of
 *                       padding groups are zero.
 *   ptqtp_packed_size = 256 + N*K_pad/2 + 4*N*K_pad/128 bytes, i.e. the Appendix B figure
 *   2*N*K*2 + (K/128)*2*N*16 bits plus the header and the K padding.
 *
 * Packed format 2 (same storage model; laid out for integer dot products: one mask yields four
 * byte-sized codes of four consecutive columns, see ptqtp_gemv):
 *   [0, 256)            header as above with format(2); the K_pad slot holds 2048 * ceil(K/2048) and the
 *                       scales_offset slot holds the bytes of one row pair over all slices.
 *   body  (at 256)      ceil(N/2) row pairs, row pair p = rows 2p and 2p+1 (a missing row 2p+1 is stored
 *                       as trit 0 with scales 0), times ceil(K/2048) slices, slice s covering columns
 *                       2048 s .. min(K, 2048 (s+1)) - 1.  Slice-major: the slice units of slice 0 for row pairs
 *                       0, 1, 2, ... lie one after the other, then those of slice 1, and so on (a kernel that
 *                       walks the rows of one slice reads one contiguous run).  A slice unit, with A =
 *                       columns/64 lane blocks:
 *                         codes   4 * A atoms of 16 bytes; atom (i, l), i = 0..3, l = 0..A-1, at byte
 *                                 16 * (i * A + l), covers the 16 columns 2048 s + 64 l + 16 i + e, e = 0..15,
 *                                 one byte per column (byte e): bits [1:0] = code of (row 2p, plane 1),
 *                                 [3:2] = (row 2p, plane 2), [5:4] = (row 2p+1, plane 1),
 *                                 [7:6] = (row 2p+1, plane 2); code q = trit + 1 in {0,1,2}.
 *                         scales  A/2 quads of 8 bytes at byte 64 * A, one per 128-column group in column
 *                                 order: fp16 alpha1[2p], alpha2[2p], alpha1[2p+1], alpha2[2p+1].
 *                         the unit is zero-padded to a multiple of 16 bytes (only when K/128 is odd).
 *                       A full slice unit is 2048 + 128 = 2176 bytes.
 *   ptqtp_packed_size = 256 + ceil(N/2) * (K + K/16 rounded up per unit) bytes; for even N and K % 256 == 0
 *   exactly the Appendix B figure plus the header.
 *
 * Packed format 3 (same storage model; the code bytes of format 2 laid out in the operand order of the int8
 * warp-level matrix instruction, so that the batch-1 kernel decodes with three masks per code word):
 *   [0, 256)            header as above with format(3); the K_pad slot holds 512 * ceil(K/512) and the
 *                       scales_offset slot holds the bytes of one tile (4352).
 *   body  (at 256)      tiles of 8 row pairs (16 rows) x 512 columns (four 128-column groups), 4352 bytes each,
 *                       superblock-major: tile (sb, rb) -- columns 512 sb .., row pairs 8 rb .. -- at byte
 *                       256 + (sb * ceil(ceil(N/2)/8) + rb) * 4352, so the tiles of one 512-column superblock for
 *                       consecutive row blocks are contiguous.  Rows >= N and columns >= K are stored as trit 0
 *                       with scales 0.  A tile:
 *                         codes   8 chunks of 512 bytes; chunk c holds for lane l = 4 g + t (g = 0..7 the row pair
 *                                 within the tile, t = 0..3) 16 bytes at 512 c + 16 l = four words (s, h) at byte
 *                                 8 s + 4 h; byte e of word (s, h) is the column byte (as in format 2) of row pair
 *                                 8 rb + g and column 512 sb + 128 (2 h + t / 2) + 8 (2 c + s) + 4 (t % 2) + e.
 *                         scales  32 quads of 8 bytes at byte 4096 + 8 l: fp16 alpha1[2p], alpha2[2p], alpha1[2p+1],
 *                                 alpha2[2p+1] of row pair p = 8 rb + g and group 4 sb + t.
 *   ptqtp_packed_size = 256 + ceil(ceil(N/2)/8) * ceil(K/512) * 4352 bytes; for N % 16 == 0 and K % 512 == 0
 *   exactly the Appendix B figure plus the header.
 */
#ifndef PTQTP_H
#define PTQTP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define PTQTP_API __attribute__((visibility("default")))
#else
#define PTQTP_API
#endif

typedef enum {
    PTQTP_OK = 0,
    PTQTP_ERR_NULL = -1,    /* a required pointer is NULL                                   */
    PTQTP_ERR_SHAPE = -2,   /* N <= 0, K <= 0, K % 128 != 0, group != 128, M out of range   */
    PTQTP_ERR_ALIGN = -3,   /* a device pointer is not 16-byte aligned                      */
    PTQTP_ERR_SIZE = -4,    /* packed buffer smaller than ptqtp_packed_size                 */
    PTQTP_ERR_TRIT = -5,    /* a plane entry outside {-1,0,1} (reported through dev_status) */
    PTQTP_ERR_FORMAT = -6,  /* bad magic / version / shape in a packed header               */
    PTQTP_ERR_CUDA = -7,    /* a CUDA runtime call failed; see ptqtp_last_cuda_error        */
    PTQTP_ERR_CONFIG = -8   /* an expert launch configuration is not supported              */
} ptqtp_status;

typedef struct {
    int32_t n_out;   /* N: output features (rows of W)            */
    int32_t k_in;    /* K: input features, multiple of 128        */
    int32_t group;   /* scale group size along K; must be 128     */
    int32_t format;  /* packed format id: 1, 2 or 3               */
} ptqtp_shape;

#define PTQTP_GROUP 128
#define PTQTP_FORMAT_V1 1
#define PTQTP_FORMAT_V2 2
#define PTQTP_FORMAT_V3 3
#define PTQTP_HEADER_BYTES 256
#define PTQTP_MAX_BATCH 64
#define PTQTP_STATIC_WORKSPACE_BYTES (512 * 1024)

/* Size in bytes of the packed blob for `shape` (header and padding included); 0 on a bad shape.
 * Storage model: Appendix B "Memory Saving" (2 bits per trit, fp16 scales per group). */
PTQTP_API size_t ptqtp_packed_size(const ptqtp_shape *shape /* host */);

/* Pack planes and scales into the streaming format (hot-path step "pack"; one-time per matrix).
 * T1, T2: device int8 [N*K], entries must be in {-1,0,1}; alpha1, alpha2: device fp16 bits [N*K/128];
 * packed: device, at least ptqtp_packed_size bytes, fully overwritten; dev_status: device int32 or
 * NULL -- receives PTQTP_ERR_TRIT if an entry is out of range (that entry is stored as 0).
 * Defines the representation of Eq. 1-2 / Appendix B used by every other call. */
PTQTP_API ptqtp_status ptqtp_pack(const ptqtp_shape *shape /* host */, const int8_t *T1, const int8_t *T2,
                        const uint16_t *alpha1, const uint16_t *alpha2, void *packed,
                        size_t packed_bytes, int32_t *dev_status, void *stream);

/* Exact inverse of ptqtp_pack: recovers the int8 planes and the fp16 scale bit patterns.
 * dev_status (device int32 or NULL) receives PTQTP_ERR_FORMAT if the blob's header does not match
 * `shape`; outputs are then unspecified. */
PTQTP_API ptqtp_status ptqtp_unpack(const ptqtp_shape *shape /* host */, const void *packed, size_t packed_bytes,
                          int8_t *T1, int8_t *T2, uint16_t *alpha1, uint16_t *alpha2,
                          int32_t *dev_status, void *stream);

/* Batch-1 decode layer y = alpha1 (.) (T1 x) + alpha2 (.) (T2 x) (Eq. 1-2 with Sec. 2.3 groups;
 * Sec. 4: additions/subtractions of x, one scale multiply per group and plane).
 * packed: device blob from ptqtp_pack (its header is not re-read; `shape` is trusted);
 * x: device fp16 [K]; y: device fp16 [N], fully overwritten.  x and y must not alias packed
 * (see also ptqtp_set_overlap).
 * Arithmetic, format 1: fp16 x times codes, fp32 accumulators, fp32 scale epilogue.
 * Arithmetic, format 2: x is turned into 16-bit block fixed point per 64 columns (exact for values within
 * 2^-5 of the block maximum, otherwise rounded to 2^-16 of it), sign-select sums are exact int32, the
 * scale epilogue and the sums over groups are fp32.  Arithmetic, format 3: x is turned into 15-bit block fixed
 * point per 128-column group (rounded to 2^-14 of the group maximum), the sign-select sums are contracted by
 * int8 warp-level matrix instructions and are exact int32, the scale epilogue and the sums over groups are fp32.
 * One rounding to fp16 at the store in all three.  Non-finite x gives unspecified y. */
PTQTP_API ptqtp_status ptqtp_gemv(const ptqtp_shape *shape /* host */, const void *packed, size_t packed_bytes,
                        const uint16_t *x, uint16_t *y, void *stream);

/* ptqtp_gemv with a gated pair epilogue, for the MLP of the LLaMA / Qwen models the paper quantises
 * (down(silu(gate(x)) * up(x)); the paper's layer, Eq. 1-2, is what yields gate(x) and up(x)).  The caller packs
 * ONE matrix of N rows (N even) that holds the gate and up projections interleaved by rows: row 2i = gate row i,
 * row 2i+1 = up row i.  With t = the layer's N fp32 row sums (before any rounding to fp16),
 *     y[i] = silu(t[2i]) * t[2i+1],   silu(g) = g / (1 + exp(-g)),   i < N/2,
 * rounded once to fp16.  y: device fp16 [N/2].  Formats 2 and 3 (PTQTP_ERR_CONFIG for format 1); PTQTP_ERR_SHAPE for
 * odd N.  Everything else as ptqtp_gemv (same kernel: only its final store differs). */
PTQTP_API ptqtp_status ptqtp_gemv_swiglu(const ptqtp_shape *shape /* host */, const void *packed, size_t packed_bytes,
                               const uint16_t *x, uint16_t *y, void *stream);

/* Several matrices that share their input in ONE launch: y[j] = layer_j(x) for j < count, 1 <= count <= 4 -- the
 * q, k and v projections of an attention block, or the gate and up projections of an MLP (Eq. 1-2 per matrix; the
 * paper reports decode speed for the model as a whole, Sec. 4 "End-to-End Speed", where these share x).  The blobs
 * are packed separately (format 3 each, PTQTP_ERR_CONFIG otherwise) and need only agree in K (PTQTP_ERR_SHAPE
 * otherwise).  shapes, packed, packed_bytes, y: host arrays of `count` entries; packed[j], x, y[j]: device.
 * x is fetched, converted and (under overlap level 2) verified once; every y[j] holds exactly the bits that
 * ptqtp_gemv gives for that matrix alone.
 * epilogue: PTQTP_EPILOGUE_NONE, or PTQTP_EPILOGUE_GATED_PAIR for count == 2 and equal N: matrix 0 is the gate,
 * matrix 1 the up projection, and ONE output y[0][i] = silu(t0[i]) * t1[i] (t = the fp32 row sums before any
 * rounding, silu(g) = g / (1 + exp(-g))) is written, rounded once to fp16; y[1] is ignored and may be NULL. */
#define PTQTP_EPILOGUE_NONE 0
#define PTQTP_EPILOGUE_GATED_PAIR 1
PTQTP_API ptqtp_status ptqtp_gemv_multi(int32_t count, const ptqtp_shape *shapes /* host */,
                              const void *const *packed /* host array */, const size_t *packed_bytes /* host */,
                              const uint16_t *x, uint16_t *const *y /* host array */, int32_t epilogue,
                              void *stream);

/* Small-batch variant: Y[m,:] = layer(X[m,:]) for m < M, 1 <= M <= PTQTP_MAX_BATCH.
 * X: device fp16 [M*K] row-major; Y: device fp16 [M*N] row-major.  Same definition per row of X.
 * Format 2, M >= 2: the planes are contracted on the tensor cores with int8 warp MMAs against 15-bit
 * block-fixed-point activations (blocks of 128 columns), exact int32 sums, fp32 scale epilogue.  M = 2..4 take
 * one pass over the planes at about the cost of a batch-1 call (the activations stay in registers); larger M
 * take one such pass per four rows (ptqtp_gemm_skinny_ws reads the planes once for any M).  When four rows of x
 * leave no room in shared memory (very long K) the passes take three or two rows, or one row on the batch-1
 * kernel.  M = 1 runs the batch-1 kernel.  Format 3, few rows: the same tiles and decode as its batch-1 kernel, with
 * the MMA columns holding two or four batch rows instead of the four scale groups (two or four times the
 * tensor-core work of one row, the same masks and the same stream of tiles); M = 2 takes one pass at about 1.3
 * times the cost of a batch-1 call, larger M take a pass per four rows (two when four rows of x leave no room in
 * shared memory).  Format 3, more rows (from M = 5 to about 20, later for small matrices: the library compares the
 * measured costs of both): one pass over the planes for all rows on the tcgen05 tensor cores -- the codes
 * are decoded to fp16 trits in tensor memory (the A operand), the activations are the fp16 B operand as given (no
 * quantisation), the sums of a scale group accumulate in fp32 in tensor memory and get the fp32 scale epilogue;
 * matrices with few rows split K over a thread-block cluster and add the partial sums in rank order
 * (reproducible).  Format 1 is a batch-1 layout: M > 1 returns PTQTP_ERR_CONFIG. */
PTQTP_API ptqtp_status ptqtp_gemm_skinny(const ptqtp_shape *shape /* host */, const void *packed,
                               size_t packed_bytes, int32_t m, const uint16_t *X, uint16_t *Y,
                               void *stream);

/* ptqtp_gemm_skinny on format 3 with the kernel chosen by the caller (tuning and tests; PTQTP_ERR_CONFIG for the
 * other formats).  path: 0 = library choice, 5 = passes of up to four rows on the warp-MMA kernel, 6 = the tcgen05
 * kernel (all M rows in one pass over the planes; fp16 trits from tensor memory against the fp16 activations, fp32
 * accumulators in tensor memory, fp32 scale epilogue).  k_split (path 6): CTAs of a cluster that share the columns
 * of a block of 128 rows: 1, 2, 4 or 8; 0 = library choice.  Same result definition as ptqtp_gemm_skinny. */
PTQTP_API ptqtp_status ptqtp_gemm_skinny_cfg(const ptqtp_shape *shape /* host */, const void *packed, size_t packed_bytes,
                                   int32_t m, const uint16_t *X, uint16_t *Y, int32_t path, int32_t k_split,
                                   void *stream);

/* Small-batch variant with a caller-provided workspace (format 2 only; PTQTP_ERR_CONFIG for format 1).
 * Same result definition as ptqtp_gemm_skinny.  The workspace (device, 16-byte aligned, at least
 * ptqtp_gemm_skinny_workspace_size(shape, m) bytes, contents irrelevant on entry, clobbered on return) holds X
 * converted once to block fixed point; with it the packed planes are read from HBM exactly once for any M and
 * K, where ptqtp_gemm_skinny needs several passes when M or K is large.  Two kernels are enqueued on `stream`.
 * Calls that share a workspace must not overlap on the GPU.  ptqtp_gemm_skinny_workspace_size returns 0 for a
 * bad shape, formats 1 and 3 (the workspace kernels read format 2) or M out of range.  (Small-batch use of the layer of Eq. 1-2; the paper measures batch 1.) */
PTQTP_API size_t ptqtp_gemm_skinny_workspace_size(const ptqtp_shape *shape /* host */, int32_t m);
PTQTP_API ptqtp_status ptqtp_gemm_skinny_ws(const ptqtp_shape *shape /* host */, const void *packed, size_t packed_bytes,
                                  int32_t m, const uint16_t *X, uint16_t *Y, void *workspace,
                                  size_t workspace_bytes, void *stream);

/* ptqtp_gemm_skinny_ws for callers that cannot hand over a workspace.  (The paper has no counterpart: this
 * entry point exists for the library's users, not for the method.)
 * Who needs it: code that runs where device memory cannot be allocated -- a plug-in or C caller inside a host
 * process whose framework already owns all of the GPU's memory through its own pool and exposes no allocator,
 * code on a latency-critical decode path where cudaMalloc/cudaFree would stall the whole device, and code
 * that must not call allocating CUDA routines at all at that point (for instance while other threads are
 * capturing streams).  The workspace is a fixed array of PTQTP_STATIC_WORKSPACE_BYTES (512 KiB) in device
 * memory that belongs to the library: every GPU that loads the library carries it until the process exits.
 * This call never calls cudaMalloc, cudaFree or any allocating library routine; the caller still owns
 * packed, X and Y.
 * Limits: the (K, M) pair must satisfy ptqtp_gemm_skinny_workspace_size(shape, m) <=
 * PTQTP_STATIC_WORKSPACE_BYTES (e.g. M <= 8 up to K = 28672, M <= 16 up to K = 14336, M <= 64 up to K = 3072);
 * otherwise PTQTP_ERR_SIZE is returned and nothing is launched.  Format 2 only (PTQTP_ERR_CONFIG for format 1).
 * The first call on each device looks up the array's device address (with that device current, no
 * allocation); make that first call outside any stream capture.
 * All calls on a device share the one array.  It keeps the previous call's contents; each call rewrites every
 * byte it later reads (padding included), so stale contents are harmless, but two calls that overlap on the
 * GPU (different streams, or the same call from two threads) race on it: serialise them. */
PTQTP_API ptqtp_status ptqtp_gemm_skinny_static(const ptqtp_shape *shape /* host */, const void *packed,
                                      size_t packed_bytes, int32_t m, const uint16_t *X, uint16_t *Y,
                                      void *stream);

/* Progressive trit-plane decomposition on the GPU: W [n, k] (device, fp32, row-major) -> planes T1, T2 (device int8
 * [n*k], entries in {-1,0,1}) and scales alpha1, alpha2 (device fp16 bits [n*k/group]) with
 * W ~ alpha1 (.) T1 + alpha2 (.) T2 per group-row -- the step before ptqtp_pack.  Algorithm 1 (group-rows, sweeps,
 * stop when the largest change of a scale pair over all group-rows is below eps or after t_max sweeps) with the
 * inner formulas of Algorithm 2 and Appendix C: initial planes sign(w) (0 -> +1), alpha = (1, 1), lambda = 1e-8;
 * ridge solve of Eq. 3-5 by the explicit 2 x 2 inverse; kappa = ||A||_F ||A^-1||_F (Eq. 6), and when kappa >= 1e6
 * lambda <- min(lambda sqrt(kappa / 1e6), 1), used by the same sweep's solve; per element the pair in {-1,0,1}^2
 * of smallest squared error, equal errors resolved towards fewer non-zeros, then towards plane 1.  The returned
 * iterate is (alpha_t, T_t) of the last sweep, without a refit.  canonicalize != 0: afterwards, per group-row and
 * without changing alpha1 T1 + alpha2 T2, both scales are made non-negative (flipping plane and scale) and ordered
 * alpha1 >= alpha2 (exchanging the planes).  The scales are rounded to fp16 once, at the end.
 * Arithmetic: IEEE double precision, every operation rounded on its own, sums in column order: a run is
 * reproducible bit for bit.  group: 1..PTQTP_DECOMPOSE_MAX_GROUP, k % group == 0 (ptqtp_pack needs group = 128);
 * t_max: 1..PTQTP_DECOMPOSE_MAX_SWEEPS (the paper uses 50, eps = 1e-4).
 * workspace: device, 16-byte aligned, ptqtp_decompose_workspace_size bytes, contents irrelevant on entry.  On
 * return (after syncing) it holds, at the offsets given by ptqtp_decompose_layout: int32 sweeps run; per sweep
 * t = 1..sweeps the largest change of a scale pair (f64 at delta_offset + 8 t) and the total squared error after the
 * sweep (f64 at error_offset + 8 (t - 1)); per group-row the unrounded scales and lambda (f64).
 * 2 t_max + 2 small kernels are enqueued on `stream`; no synchronisation. */
#define PTQTP_DECOMPOSE_MAX_GROUP 256
#define PTQTP_DECOMPOSE_MAX_SWEEPS 1000
typedef struct {
    size_t sweeps_offset;   /* int32 */
    size_t delta_offset;    /* f64 [t_max + 1], entry t for sweep t */
    size_t error_offset;    /* f64 [t_max] */
    size_t alpha1_offset;   /* f64 [n * k / group] */
    size_t alpha2_offset;   /* f64 [n * k / group] */
    size_t lambda_offset;   /* f64 [n * k / group] */
    size_t total_bytes;
} ptqtp_decompose_offsets;
PTQTP_API size_t ptqtp_decompose_workspace_size(int32_t n, int32_t k, int32_t group, int32_t t_max);
PTQTP_API ptqtp_status ptqtp_decompose_layout(int32_t n, int32_t k, int32_t group, int32_t t_max,
                                    ptqtp_decompose_offsets *out /* host */);
PTQTP_API ptqtp_status ptqtp_decompose(const float *W, int32_t n, int32_t k, int32_t group, int32_t t_max, double eps,
                             int32_t canonicalize, int8_t *T1, int8_t *T2, uint16_t *alpha1, uint16_t *alpha2,
                             void *workspace, size_t workspace_bytes, void *stream);

/* End-to-end convenience for callers holding activations on the host: copies x_host [K] (host,
 * ideally pinned) to x_dev, runs ptqtp_gemv and delivers y in y_host [N]; everything is enqueued on
 * `stream`, no synchronisation: y_host is valid once the stream has reached this point.  x_dev [K] and
 * y_dev [N] are caller-owned device staging buffers.  When y_host is pinned, 16-byte aligned memory that the
 * device can address (format 2), the kernel stores y there directly and y_dev is left untouched; otherwise
 * y is computed into y_dev and copied to y_host. */
PTQTP_API ptqtp_status ptqtp_gemv_host(const ptqtp_shape *shape /* host */, const void *packed, size_t packed_bytes,
                             const uint16_t *x_host, uint16_t *y_host, uint16_t *x_dev, uint16_t *y_dev,
                             void *stream);

/* Expert entry point: ptqtp_gemv with an explicit launch configuration, for tuning and tests.
 * rows_per_warp in {1,2,4}; k_split (warps of a CTA sharing a row, splitting K; must divide
 * K_pad/1024) in {1,2,4,8}; ctas_per_sm >= 1 bounds the persistent grid (grid = min(tiles,
 * ctas_per_sm * SM count)); depth = 128-bit loads per row kept in flight per lane (1,2,4,8; not
 * every combination with rows_per_warp is built); 0 in any of these selects the library's own choice.
 * arith: accumulation of the sign-selected activations -- 0 = fp32 accumulator fed by mixed-precision
 * FMAs (fp16 operands), 1 = fp16x2 chains of 4 flushed into fp32, 2 = chains of 8, -1 = library choice.
 * PTQTP_ERR_CONFIG if the combination is not built.
 * For a format-2 blob the arguments mean: arith = -1 (library choice), 3 (masks and integer dot products on
 * the CUDA cores) or 4 (int8 tensor-core MMAs, the kernel behind ptqtp_gemm_skinny for two to four rows).
 * arith 3: rows_per_warp = slice units per bulk copy (1, 2 or 4; 0 = 2, or 1 when x is long); k_split = warps
 * per CTA (1..16 / ctas_per_sm, 0 = auto: 4 to 8, so that the CTAs of several consecutive launches fit on an SM
 * together; 16 serves a call that runs alone best); ctas_per_sm = CTAs of this launch per SM (1..4, 0 = 1);
 * depth = copies in flight per warp (2, 3, 4, 6, 8; 0 = 2).  arith 4: rows_per_warp must be 0; k_split = warps
 * per CTA (4, 8 or 16, 0 = auto); ctas_per_sm 1 or 2 (0 = 1); depth = stages (four slice units each) per team of
 * four warps (2..8, 0 = auto).  A configuration that does not fit in shared memory gives PTQTP_ERR_CONFIG.
 * For a format-3 blob: arith = -1 or 5; rows_per_warp = tiles per bulk copy (1 or 2, 0 = library choice);
 * k_split = warps per CTA (1..16 / ctas_per_sm, 0 = library choice, -1 = as many as have work: for a call that runs
 * alone); ctas_per_sm = CTAs of this launch per SM (1..4, 0 = 1); depth = copies in flight per warp (2, 3, 4, 6;
 * 0 = library choice). */
PTQTP_API ptqtp_status ptqtp_gemv_cfg(const ptqtp_shape *shape /* host */, const void *packed, size_t packed_bytes,
                            const uint16_t *x, uint16_t *y, int32_t rows_per_warp, int32_t k_split,
                            int32_t ctas_per_sm, int32_t depth, int32_t arith, void *stream);

/* Parse the 256-byte header of a packed blob that was copied to the host (e.g. read from a file).
 * Fills *shape and returns PTQTP_OK, or PTQTP_ERR_FORMAT / PTQTP_ERR_SIZE / PTQTP_ERR_NULL. */
PTQTP_API ptqtp_status ptqtp_parse_header(const void *header_host, size_t bytes, ptqtp_shape *shape /* host */);

/* Human-readable name of a status code (static storage, never NULL). */
PTQTP_API const char *ptqtp_status_string(ptqtp_status status);

/* The cudaError_t (as int) behind the calling thread's most recent PTQTP_ERR_CUDA, else 0. */
PTQTP_API int ptqtp_last_cuda_error(void);

/* Device-side health of the kernels that stream the packed planes with bulk copies (batch 1 of formats 2 and 3,
 * and the small-batch kernel for two to four rows) on the current device.  They wait for each copy with a bounded
 * number of polls; if a wait ever gives up, the kernel
 * writes NaN to the rows it could not finish, records PTQTP_ERR_CUDA in a device word and still terminates.
 * This call enqueues a copy of that word (0 = healthy) to *status_host on `stream`; read it after syncing. */
PTQTP_API ptqtp_status ptqtp_kernel_status(int32_t *status_host /* host */, void *stream);

/* Reset that device word to 0 (enqueued on `stream`): the word is only ever set by the kernels, so after a
 * reported failure it keeps its value until this call. */
PTQTP_API ptqtp_status ptqtp_kernel_status_clear(void *stream);

/* Number of polls after which a bounded wait for a bulk copy gives up (process-wide, default 2^22, at least 1;
 * returns the old value).  A poll takes from tens of nanoseconds to a few microseconds. */
PTQTP_API int ptqtp_set_wait_limit(int polls);

/* Test hook for the give-up path of the bounded waits: each of the next `launches` format-3 batch-1 launches
 * announces, on one mbarrier of its first CTA, 16 bytes more than the copy brings, so that wait runs out after
 * ptqtp_set_wait_limit polls: the affected rows come out as NaN and ptqtp_kernel_status reports PTQTP_ERR_CUDA.
 * Every copy still lands and the kernel ends normally.  Not for production use. */
PTQTP_API void ptqtp_test_fail_next_wait(int launches);

/* Overlap of consecutive GEMV calls on one stream (process-wide level, default 0; returns the old level).
 * Level 0 (default): plain launches; every buffer, `packed` included, follows stream order.  Levels 1 and 2 are
 * an opt-in for callers whose packed blobs are immutable while GEMV calls are in flight (the decode case).
 * Level 1: the GEMV kernels of formats 2 and 3 are launched with programmatic stream
 * serialization: a call may begin reading its `packed` blob while the kernel directly before it on the
 * stream is still draining; x is used and y written only after all earlier work on the stream has completed,
 * so stream order holds for them.  Consequence for the caller: the packed blob of a call must be complete
 * before the kernel directly ahead of the call on its stream ends -- it must not be the output buffer of that
 * kernel.  ptqtp_pack is exempt (the first GEMV call after a ptqtp_pack on the same stream is a plain launch),
 * and so are copies (cudaMemcpyAsync and the like are not kernels).  Works inside CUDA graph capture.
 * Level 2 adds speculative execution: the kernel reads x at once and computes everything into shared memory
 * while earlier work of the stream may still be running, then waits for that work, reads x again and compares
 * it bit by bit with its first read; y is written only after that, and if a single bit of x differed the whole
 * computation is repeated from the second read.  Results are identical to level 1 in every case.  It pays when
 * x was finished before the call directly ahead of this one started (k and v after q, up after gate, any call
 * behind work that is not a GEMV of this library) and costs a second pass over the matrix when it was not (y of
 * the GEMV directly ahead used as x). */
PTQTP_API int ptqtp_set_overlap(int level);

/* Library version: major*10000 + minor*100 + patch. */
PTQTP_API int ptqtp_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PTQTP_H */
