/*
 * libtsvd -- the Ternary-SVD parameterised linear map on one NVIDIA B200 (sm_100a).
 *
 *     y = U ( diag(S) ( V x ) )
 *
 * U [M,K] and V [K,N] hold only -1, 0, +1; S is a real vector of length K; x is a
 * batch of B activation columns.  This is the inference-time form of the paper's
 * TSVD layer (Section "Truncated SVD in Network Compression", Eq. 1-2 and the
 * display that follows them; Section "Ternary SVD"), whose cost the paper counts
 * as r*K*(M+N) additions and K multiplications per column (supplement, Table S1).
 *
 * Plain C ABI: pointers and sizes only.  Every call returns a status; nothing is
 * thrown across the boundary; arguments are validated on the host before any
 * kernel is launched.  There is no CPU implementation behind these calls: without
 * a CUDA device they return TSVD_E_CUDA.
 *
 * Arithmetic of the fast kernels (tensor-core, decode and index-list paths), which is
 * what bounds their accuracy.  Per token (the decode kernels: per token and quarter of
 * the columns, from three tokens and 1024 columns on), the activations are rounded once to a
 * multiple of 2^(E-22) (bf16 activations; 2^(E-30) with TSVD_FLAG_WIDE_X) or 2^(E-30)
 * (fp32 activations), where 2^E is the power of two just above the token's largest
 * magnitude; int8 activations are used as they are.  From there the V-stage is exact
 * integer arithmetic (z = V x is bit-exact for int8 activations), t = S * z is one fp32
 * product per rank component, t is rounded likewise to a multiple of 2^(E_t-30), the
 * U-stage is exact again, and y is rounded once to its output type.  Consequences:
 *   - activations must be finite (NaN and Inf are not detected; y is then unspecified);
 *   - entries far below a token's largest magnitude lose bits: an entry 2^-s of the
 *     largest keeps 22-s (30-s) bits.  With the bulk of a bf16 token within 2^8 of its
 *     largest entry (2^16 with TSVD_FLAG_WIDE_X and for fp32), every output meets
 *     |y - y_exact| <= 1e-2 |y_exact| + 1e-3 at the value scales of transformer
 *     activations; a forward that meets a token outside that range reports
 *     TSVD_E_RANGE through tsvd_last_status (see there), and the CUDA-core path
 *     (TSVD_FLAG_PATH_SIMPLE: fp32 partial sums per 64 columns, fp64 across) has no
 *     such limit;
 *   - a token whose largest magnitude is below 2^-90 is scaled as if it were 2^-90,
 *     so it loses bits, and below about 2^-120 it is treated as zero.
 */
#ifndef TSVD_H
#define TSVD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tsvd_handle_s* tsvd_handle_t; /* opaque; owns device memory on one GPU */

/* storage type of the activations x */
typedef enum { TSVD_F32 = 0, TSVD_BF16 = 1, TSVD_I8 = 2 } tsvd_dtype_t;

typedef enum {
    TSVD_OK = 0,
    TSVD_E_NULL = 1,    /* a required pointer is NULL                              */
    TSVD_E_SHAPE = 2,   /* a size is < 1, a leading dimension is too small, ...    */
    TSVD_E_VALUE = 3,   /* an entry of U or V is outside {-1,0,+1}                  */
    TSVD_E_DTYPE = 4,   /* unknown dtype or unsupported flag combination           */
    TSVD_E_ALIGN = 5,   /* a pointer or leading dimension breaks the stated rule   */
    TSVD_E_CUDA = 6,    /* a CUDA runtime call failed (or there is no device)      */
    TSVD_E_TIMEOUT = 7, /* a bounded device-side wait gave up                      */
    TSVD_E_NOMEM = 8,   /* host or device allocation failed                        */
    TSVD_E_TOOBIG = 9,  /* request exceeds a fixed capacity (tsvd_forward_static, TSVD_MAX_CONTRACTION) */
    TSVD_E_RANGE = 10,  /* tsvd_last_status only: a token's dynamic range exceeded what the
                           fixed-point digits resolve (see the note on arithmetic above)   */
    TSVD_E_INTERNAL = 11 /* tsvd_last_status only, builds with -DTSVD_CHECK_BOUNDS: a kernel found
                           one of its ring or tile indices outside its range              */
} tsvd_status_t;

/* Longest contraction (N and K) a handle may have: the digit sums of a row are combined in
 * 32-bit integers, |sum| <= 128 * 257 * columns, which stays below 2^31 up to here. */
#define TSVD_MAX_CONTRACTION 65280

/* flags of tsvd_forward_ex */
#define TSVD_FLAG_OUT_F32 0x1u      /* write y as fp32 even for bf16 activations            */
#define TSVD_FLAG_PATH_SIMPLE 0x10u /* force the CUDA-core reference kernels               */
#define TSVD_FLAG_PATH_DECODE 0x20u /* force the decode kernels (B <= TSVD_DECODE_MAX_B)    */
#define TSVD_FLAG_PATH_TENSOR 0x40u /* force the tcgen05 tensor-core kernels               */
#define TSVD_FLAG_PATH_INDEX 0x80u  /* run the index-list kernels (see TSVD_PACK_INDEX_LISTS) */
#define TSVD_FLAG_PATH_MASK 0xF0u   /* at most one of the four may be set                     */
/* bf16 activations as four signed 8-bit digits (30 bits of the token's range) instead of
 * three (22 bits): for tokens with outliers up to 2^16 times their bulk.  The V-stage of the
 * tensor-core path then executes 4/3 of the operations; no effect on fp32 and int8. */
#define TSVD_FLAG_WIDE_X 0x200u
/* The decode kernels (two launches, one per stage; each CTA streams 32 rows of the packed
 * codes against fixed-point digits of the stage's input held in shared memory) serve batches
 * of at most this many tokens.  They are the default up to four tokens, and up to eight where
 * both contractions have 1024 columns or more; beyond that, up to 32 tokens, the default is a
 * pair of cluster kernels of the tensor-core path (TSVD_FLAG_PATH_TENSOR; one launch per stage,
 * contractions of up to 4096 columns), and the tile kernels of that path otherwise.
 * Forcing the decode kernels for a larger batch, or for a contraction too long for the digits to fit in
 * shared memory, returns TSVD_E_TOOBIG (one and two tokens fit at any supported length, four up to about
 * 40,000 columns, sixteen up to about 12,000; nine to sixteen tokens also need 1024 columns or more in
 * both stages). */
#define TSVD_DECODE_MAX_B 16
/* the index-list kernels serve at most this many tokens */
#define TSVD_INDEX_MAX_B 4
/* Test hook for the bounded device-side waits: the V-stage kernel of the tensor-core path
 * withholds the activation digits (B > 64: its copy producer; fewer tokens: the converting warps
 * never declare them ready), so every wait on them runs out (after a few
 * milliseconds instead of the usual ~2 s); all CTAs then leave through their normal exit,
 * y is unspecified, and tsvd_last_status reports TSVD_E_TIMEOUT.  No fault, no hang: the
 * context and the handle stay usable. */
#define TSVD_FLAG_TEST_STALL 0x100u

/* tsvd_pack flag: also keep U and V as index lists -- per row the list of its nonzeros, 16
 * bits each, (column << 1) | (1 for -1) -- for forwards of up to TSVD_INDEX_MAX_B tokens with
 * TSVD_FLAG_PATH_INDEX.  The paper calls 2 bits per element a redundant code for sparse U
 * and V (Section "Connection with BNN and What Next"); this form is the smaller one below a
 * nonzero rate of 1/8 and its forward does exactly the additions of Table S1, one per nonzero.
 * It is run on request only (never chosen by default); a forward that asks for it on a handle
 * packed without it, or for more tokens, returns TSVD_E_TOOBIG. */
#define TSVD_PACK_INDEX_LISTS 0x1u
#define TSVD_INDEX_MAX_COLUMNS 32768 /* a column index has 15 bits */

/*
 * tsvd_pack -- store U and V in a 2-bit sign/nonzero form (two bits per entry are what
 * the paper says a ternary matrix needs, Section "Connection with BNN and What Next";
 * the split U = U+ - U-, V = V+ - V- of the same section) and copy S.
 *
 *   U  host, int8 [M,K] row-major        V  host, int8 [K,N] row-major
 *   S  host, float [K] (any finite values: negative, zero, unsorted are all fine)
 *   flags  0, or TSVD_PACK_INDEX_LISTS
 *   out    receives the handle; device memory lives on the current CUDA device
 *
 * The inputs are copied; the caller keeps ownership of U, S, V.  Any M,K,N >= 1:
 * ragged sizes are padded with zero entries, which contribute nothing.
 * Synchronous.  Errors: E_NULL, E_SHAPE, E_VALUE (nothing is kept), E_NOMEM, E_CUDA,
 * E_DTYPE (unknown flag), E_TOOBIG (index lists asked for with N or K above
 * TSVD_INDEX_MAX_COLUMNS).
 */
tsvd_status_t tsvd_pack(const int8_t* U, const float* S, const int8_t* V, int M, int K, int N,
                        unsigned flags, tsvd_handle_t* out);

/*
 * tsvd_forward -- y = U(diag(S)(V x)) for B columns (display after Eq. 2):
 * V-stage additions, K multiplications by S, U-stage additions (Table S1).
 *
 *   x  device; column b is the N contiguous values at x + b*N (token-major)
 *   y  device; column b is the M contiguous values at y + b*M
 *      y is fp32 for TSVD_F32 and TSVD_I8 activations, bf16 (round-to-nearest-even
 *      from the fp32 result) for TSVD_BF16
 *   stream  a cudaStream_t (NULL = default stream); the call is asynchronous
 *
 * x and y stay owned by the caller and must be 16-byte aligned.  The handle's
 * scratch memory is shared by all calls on it: calls on one handle must be
 * ordered on one stream (or otherwise serialised).  Scratch grows on the first call
 * with a larger B (that call synchronises the device once) unless tsvd_reserve has
 * sized it beforehand.  x must be finite (see the note on arithmetic at the top).
 * Errors: E_NULL, E_SHAPE (B < 1), E_DTYPE, E_ALIGN, E_NOMEM, E_CUDA.
 */
tsvd_status_t tsvd_forward(tsvd_handle_t h, const void* x, void* y, int B, tsvd_dtype_t dtype,
                           void* stream);

/*
 * tsvd_forward_ex -- tsvd_forward with leading dimensions, flags and the V-stage
 * result exposed (Table S1, row "V(.)").
 *
 *   ldx >= N, ldy >= M   in elements; column b at x + b*ldx, y + b*ldy
 *   z_out  optional device buffer [B][K] receiving V x BEFORE the S scale:
 *          int32 (exact) for TSVD_I8, fp32 otherwise
 */
tsvd_status_t tsvd_forward_ex(tsvd_handle_t h, const void* x, int ldx, void* y, int ldy, int B,
                              tsvd_dtype_t dtype, unsigned flags, void* z_out, void* stream);

/*
 * tsvd_forward_v -- the first two rows of Table S1 alone: t = diag(S)(V x), fp32, for B columns.
 * The convolution forms of a TSVD layer (Section "TSVD in Convolution Layer") apply V(.) and U(.) as
 * two convolutions with the channel-wise scale between them; each of the two is this call on the
 * patches of its input (see tsvd_im2col), with the ternary matrix of that stage packed as the V of
 * a handle (S = 1 and a 1-row U of zeros for the stage that has no scale).
 *
 *   x      device, B columns at x + b*ldx (ldx >= N), 16-byte aligned, dtype as tsvd_forward
 *   t_out  device, float, column b at t_out + b*ldt (ldt >= K), 16-byte aligned
 *   flags  TSVD_FLAG_PATH_SIMPLE / _DECODE / _TENSOR, TSVD_FLAG_WIDE_X (not _INDEX, not _OUT_F32)
 * Asynchronous on `stream`; same scratch rules as tsvd_forward.
 * Errors: as tsvd_forward_ex; E_DTYPE for TSVD_FLAG_PATH_INDEX.
 */
tsvd_status_t tsvd_forward_v(tsvd_handle_t h, const void* x, int ldx, float* t_out, int ldt, int B,
                             tsvd_dtype_t dtype, unsigned flags, void* stream);

/*
 * tsvd_im2col -- the patches of an image batch, so that a convolution with a ternary kernel becomes
 * the ternary matrix product of this library (Section "TSVD in Convolution Layer": V(.) and U(.) in
 * convolution form with kernels [K1,K2], [1,1], [K1,1] or [1,K2]).
 *
 *   x    device, n_img images in NHWC layout: x[((n*H + h)*W + w)*C + c], dtype as given
 *   out  device, same dtype: row (n, ho, wo) at out + ((n*Ho + ho)*Wo + wo)*ld_out holds the k1*k2*C
 *        values x[n, ho*stride_h + a*dil_h - pad_h, wo*stride_w + b*dil_w - pad_w, c] at index
 *        (a*k2 + b)*C + c, zero where the position lies outside the image;
 *        Ho = (H + 2 pad_h - dil_h (k1-1) - 1) / stride_h + 1, Wo likewise; ld_out >= k1*k2*C
 * Asynchronous on `stream`; the caller owns both buffers.  Errors: E_NULL, E_SHAPE, E_DTYPE, E_CUDA.
 */
tsvd_status_t tsvd_im2col(const void* x, tsvd_dtype_t dtype, int n_img, int H, int W, int C, int k1, int k2,
                          int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w, void* out,
                          long long ld_out, void* stream);

/*
 * tsvd_forward_v_patches -- tsvd_im2col and tsvd_forward_v in one call, without the patch matrix: the
 * stage's tokens are the patches of the image batch at x, read in place while they are converted for the
 * tensor-core kernels (Section "TSVD in Convolution Layer": V(.) or U(.) as a convolution).  The result
 * is, bit for bit, that of tsvd_forward_v on the output of tsvd_im2col.
 *
 *   x      device, n_img NHWC images of dtype `dtype`, 16-byte aligned; C a multiple of 16
 *   geometry as tsvd_im2col; k1*k2*C must equal the handle's N; B = n_img*Ho*Wo tokens
 *   t_out  device, float, row (n, ho, wo) at t_out + ((n*Ho + ho)*Wo + wo)*ldt (ldt >= K), 16-byte aligned
 *   flags  TSVD_FLAG_WIDE_X; TSVD_FLAG_PATH_TENSOR to take the tensor-core kernels for 16 tokens and fewer
 * Asynchronous on `stream`; same scratch rules as tsvd_forward.
 * Errors: as tsvd_forward_v; E_SHAPE also when C is not a multiple of 16, when k1*k2*C != N, or when
 * the batch would not run on the tensor-core kernels (use tsvd_im2col + tsvd_forward_v there).
 */
tsvd_status_t tsvd_forward_v_patches(tsvd_handle_t h, const void* x, tsvd_dtype_t dtype, int n_img, int H, int W, int C,
                                     int k1, int k2, int stride_h, int stride_w, int pad_h, int pad_w, int dil_h,
                                     int dil_w, float* t_out, int ldt, unsigned flags, void* stream);

/*
 * tsvd_forward_host -- the same map with HOST buffers: copies x to the device, runs
 * tsvd_forward_ex, copies y (and z_out) back, and waits.  x, y, z_out are host pointers;
 * layout as tsvd_forward.  Batches of 768 tokens and more are cut into about eight chunks
 * that are pipelined over three streams of the handle (copy-in, compute, copy-out), so that
 * with pinned host memory the copies of neighbouring chunks overlap the computation; the
 * result does not depend on the chunking (tokens are independent).
 */
tsvd_status_t tsvd_forward_host(tsvd_handle_t h, const void* x, void* y, int B,
                                tsvd_dtype_t dtype, unsigned flags, void* z_out);

/*
 * tsvd_forward_static -- tsvd_forward for callers that must not allocate.
 * (The paper has no counterpart to this call: it is a deployment convenience.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a serving
 * loop whose memory budget was fixed at start-up and is audited, in a process that
 * hands the whole device to another allocator and forbids side allocations, or in
 * a latency-critical section where an allocation's implicit device synchronisation
 * is unacceptable.  tsvd_forward grows a per-handle scratch buffer with cudaMalloc
 * the first time it sees a larger batch; this call never allocates or frees: its
 * intermediate S*(V x) lives in a fixed array of TSVD_STATIC_SCRATCH_BYTES that is
 * part of the library image (every GPU that loads the library holds those bytes
 * until the process exits).
 *
 *   h, x, y, B, dtype, stream   exactly as tsvd_forward (x, y device, token-major,
 *                               16-byte aligned; y fp32, or bf16 for bf16 x)
 *
 * Limit: B * roundup(K,128) * 4 bytes must fit in TSVD_STATIC_SCRATCH_BYTES,
 * otherwise TSVD_E_TOOBIG is returned and nothing is launched.
 * First call on a device: looks up the array's device address once (with that device
 * current, which the handle already requires); make that first call before any
 * stream capture begins.
 * Sharing: there is ONE array per device, used by every handle and every call.  It
 * keeps the previous call's contents; nothing in it has to start at zero, because
 * the V-stage overwrites every element the U-stage reads.  Two calls that overlap on
 * the GPU (different streams, no ordering between them) race on it: order them.
 * Runs the CUDA-core kernels.  Errors: as tsvd_forward, plus E_TOOBIG.
 */
#define TSVD_STATIC_SCRATCH_BYTES (4u << 20)
tsvd_status_t tsvd_forward_static(tsvd_handle_t h, const void* x, void* y, int B,
                                  tsvd_dtype_t dtype, void* stream);

/*
 * tsvd_reserve -- size the handle's scratch once, so that no later tsvd_forward /
 * tsvd_forward_ex with at most B_max tokens of this dtype (any flags, any path)
 * allocates, frees or synchronises: such forwards can then be captured in a CUDA graph
 * from the first call on.  Synchronises the device if the scratch has to grow.
 * (Measurement and deployment support; the paper has no counterpart.)
 * Errors: E_NULL, E_SHAPE, E_DTYPE, E_NOMEM, E_CUDA.
 */
tsvd_status_t tsvd_reserve(tsvd_handle_t h, int B_max, tsvd_dtype_t dtype);

/*
 * tsvd_set_bias -- y = U(diag(S)(V x)) + b.  Eq. 1 of the paper is written without a bias,
 * but every layer of its architecture listing (supplement) carries one (`bias=True`); it is
 * added in fp32 to the U-stage result before the single rounding to the output type.
 *   bias  host, float [M]; copied.  NULL removes the bias again.
 * Synchronous; must not be called while a forward on this handle is in flight.
 * Errors: E_NULL (h), E_NOMEM, E_CUDA.
 */
tsvd_status_t tsvd_set_bias(tsvd_handle_t h, const float* bias);

/*
 * tsvd_ternarize -- the ternarisation T(x, theta) of Algorithm 1 (Section "Direct Transition
 * Algorithm to TSVD form"), the step that turns the singular vectors of the residual into new
 * columns of U and rows of V in Algorithm 2.  For each of n_vec vectors: the sparsest vector
 * over {-1,0,+1} whose angle to x is at most theta; it keeps sign(x) on the k largest
 * magnitudes, k the first index at which (sum of the k largest |x|) / sqrt(k) / ||x|| reaches
 * cos(theta) (sums and the comparison in double precision), and every entry whose magnitude
 * equals the k-th largest is kept with it.
 *
 *   x      device, float; vector v is the len values at x + v*ldx (ldx >= len)
 *   theta  angle in radians, 0 <= theta <= pi/2 (the paper uses 0.576)
 *   t      device, int8; receives vector v at t + v*ldt (ldt >= len)
 *   nnz    device, int [n_vec], optional: the number of nonzeros of each result, or -1 where no
 *          ternary vector lies within theta of x (Theorem 1 bounds when that can happen); the
 *          result is then all zeros
 *   stream a cudaStream_t; the call is asynchronous; the caller keeps ownership of all buffers
 * Errors: E_NULL, E_SHAPE (sizes, leading dimensions, theta out of range), E_TOOBIG (len above
 * TSVD_TERNARIZE_MAX_LEN: a vector is sorted in the shared memory of one SM), E_CUDA.
 */
#define TSVD_TERNARIZE_MAX_LEN 32768
tsvd_status_t tsvd_ternarize(const float* x, int n_vec, int len, int ldx, double theta, int8_t* t, int ldt,
                             int* nnz, void* stream);

/* Device-side status word of the forwards on this handle since the last read (read after
 * the stream has been synchronised).  Resets the word.  Returns
 *   TSVD_E_TIMEOUT if a bounded wait inside a kernel gave up (y is then unspecified), else
 *   TSVD_E_RANGE   if some token's dynamic range was wider than the fixed-point digits
 *                  resolve: while converting a stage's input the kernels sample one value
 *                  in eight, and raise this when, among at least 32 nonzero samples of a
 *                  token that one warp or one CTA converted, fewer than a quarter reach 2^12
 *                  quantisation steps (most entries then keep fewer than 12 bits; for a
 *                  normally distributed bulk this happens from an outlier of about 2^10
 *                  times the bulk's scale with three digits, 2^18 with four).  y is still
 *                  the result of the arithmetic described at the top of this file; rerun
 *                  with TSVD_FLAG_WIDE_X or TSVD_FLAG_PATH_SIMPLE if it must meet the
 *                  tolerance;
 *   TSVD_OK        otherwise. */
tsvd_status_t tsvd_last_status(tsvd_handle_t h);

/* Shapes, packed size in bytes (U and V codes plus S: the bytes a forward must
 * stream) and the measured nonzero rates r of U and V (the r of Table S1). */
tsvd_status_t tsvd_info(tsvd_handle_t h, int* M, int* K, int* N, size_t* packed_bytes,
                        double* density_u, double* density_v);

/* Bytes of the index-list form of V and of U (row pointers + 16-bit entries: what an
 * index-list forward streams); 0 for a handle packed without TSVD_PACK_INDEX_LISTS. */
tsvd_status_t tsvd_index_bytes(tsvd_handle_t h, size_t* v_bytes, size_t* u_bytes);

/* Inverse of tsvd_pack, for tests: writes the stored U [M,K], V [K,N] (int8) and
 * S [K] back to HOST buffers (any of them may be NULL). */
tsvd_status_t tsvd_unpack(tsvd_handle_t h, int8_t* U, float* S, int8_t* V);

/*
 * tsvd_plan -- which kernels a forward with these arguments would run (no launch).
 *   path  receives TSVD_FLAG_PATH_SIMPLE, _DECODE, _TENSOR or _INDEX
 *   digits_x, digits_t  receive the number of signed 8-bit digits the tensor-core and
 *   decode paths use for the activations and for S*(V x) (0 on the CUDA-core path).  Executed tensor
 *   operations per forward = 2*B*(K*N*digits_x + M*K*digits_t) on the padded shapes; the
 *   paper's own count is additions at the nonzeros only (Table S1).
 */
tsvd_status_t tsvd_plan(tsvd_handle_t h, int B, tsvd_dtype_t dtype, unsigned flags, unsigned* path,
                        int* digits_x, int* digits_t);

/*
 * Per-stage device timing (measurement support; the paper reports operation counts
 * per stage in Table S1 and no timings).
 *   mode 0  off
 *   mode 1  every forward on the handle records a CUDA-event pair on its stream around
 *           each kernel it launches (eager streams only; a pair includes the launch
 *           latency of a short kernel)
 *   mode 2  every kernel launched for the handle writes the device's nanosecond timer
 *           itself: its first CTA once its wait for the kernel before it has ended, and
 *           every warp when it finishes (the maximum is kept).  This works inside a
 *           captured CUDA graph: each captured launch owns a pair of words, which every
 *           replay overwrites.  Up to 32768 launches are recorded after the call.
 * tsvd_profile_read synchronises, then returns, per stage, the summed device time in
 * milliseconds and the number of launches (both arrays have TSVD_N_STAGES entries).  In
 * mode 1 it covers the launches since the last read and resets the sums; in mode 2 it
 * covers every launch recorded since tsvd_profile_enable, as last executed.
 *   stage 0: activations -> integer digits     stage 1: V-stage (+ S scale)
 *   stage 2: S*(V x)     -> integer digits     stage 3: U-stage
 */
#define TSVD_N_STAGES 4
tsvd_status_t tsvd_profile_enable(tsvd_handle_t h, int mode);
tsvd_status_t tsvd_profile_read(tsvd_handle_t h, float* ms_sum, unsigned* launches);

/* Number of kernels this library has launched in this process (all handles). */
unsigned long long tsvd_launch_count(void);

void tsvd_destroy(tsvd_handle_t h);
const char* tsvd_strerror(tsvd_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* TSVD_H */
