// Tensor-core path for batched forwards: both stages of y = U(diag(S)(V x)) as integer
// contractions on tcgen05 (kind::i8, int32 accumulators in tensor memory).
//
// Table S1 counts the V- and U-stage as additions only.  For a batch those additions are a
// dense contraction of a {-1,0,+1} matrix with the activations, so they are issued to the
// tensor cores with the ternary operand expanded on chip to int8 +-1/0.  To keep the
// arithmetic exact the real-valued operand is first written as a per-token fixed-point
// integer split into signed 8-bit digits (radix 256): every product and every partial sum
// is then an exact integer, the result does not depend on summation order, and the only
// roundings are the fixed-point step of the operand and the final conversion to fp32.
//
//   digitise(x)  ->  V-stage MMA  ->  epilogue: z = int * 2^e, t = S*z (the K multiplications)
//                ->  digitise(t)  ->  U-stage MMA  ->  epilogue: y = int * 2^e
//
// Batches above 64 tokens use 192-column tiles, one CTA per tile; smaller batches use 16-token
// tiles with the contraction split across CTAs (integer atomics, the last part of a tile
// finishes the stage), so that the packed codes are streamed by about one CTA per SM.
#include "digits.cuh"
#include "sm100_ptx.cuh"
#include "tsvd_internal.cuh"

namespace {

using namespace ptx;

constexpr int BLOCK_R = 128;   // ternary rows per CTA tile = MMA M
constexpr int BLOCK_C = 128;   // contraction elements per block (one 128-byte swizzle row)
constexpr int STEP_BLOCKS = 2; // blocks per pipeline step: one set of barrier handshakes covers this many
constexpr int UMMA_K = 32;     // contraction elements per kind::i8 instruction
constexpr int NT_MAX = 192;    // MMA N extent: digit rows per tile
constexpr int NP = 4;          // ring depth (steps) of the packed codes (shared memory)
constexpr int NB = 4;          // ring depth (steps) of the digit tiles (shared memory) and of the per-step barriers
constexpr int NA = 2;          // ring depth (steps) of the expanded ternary operand (tensor memory)
// tensor memory: two accumulator buffers of 192 columns, then two 64-column slots that hold
// the expanded ternary operand of a step (per block 128 rows x 128 int8 = 32 columns of 32 bits)
constexpr int TMEM_COLS = 512;
constexpr int ACC_COLS = NT_MAX;
constexpr int A_COL0 = 2 * ACC_COLS;
constexpr int A_BLOCK_COLS = BLOCK_C / 4;
constexpr int A_SLOT_COLS = STEP_BLOCKS * A_BLOCK_COLS;
static_assert(A_COL0 + NA * A_SLOT_COLS <= TMEM_COLS, "tensor memory budget");
// warp 0: digit-tile copies, 1: MMA issue, 2: packed-code copies, 3: idle,
// 4..11: expand (two groups of four that take alternate steps), 12..: epilogue (four or eight)
constexpr int EXP_GROUPS = 2;     // groups of four expander warps; group g takes steps it % EXP_GROUPS == g
constexpr int EXP_WARP0 = 4;
constexpr int EPI_WARP0 = EXP_WARP0 + 4 * EXP_GROUPS;
// Epilogue warps: one per 32 tensor-memory lanes, times EPIW / 4 shares of a tile's tokens.  Eight
// keep up with tiles of a few contraction blocks; four are enough when a tile's MMAs (384 clocks
// per block) outlast the drain of its TOK tokens per row (about 100 clocks each with four warps),
// and they leave more issue slots to the expanders meanwhile.
constexpr int EPI_WARPS_MAX = 8;
__host__ __device__ constexpr bool four_epilogue_warps(int kb_tile, int tok) { return 3 * kb_tile >= tok; }
__host__ __device__ constexpr int gemm_threads(int epiw) { return 32 * (EPI_WARP0 + epiw); }

// tokens per tile for nd digits: the MMA N extent is nd * tokens = 192 for every nd
__host__ __device__ constexpr int tokens_per_tile(int nd) { return 192 / nd; }

constexpr int P_TILE_BYTES = BLOCK_R * BLOCK_C / 4;      // packed codes of that tile, 4 KiB
constexpr int B_TILE_BYTES_MAX = NT_MAX * BLOCK_C;       // digit rows, 24 KiB
constexpr int B_SLOT_BYTES = STEP_BLOCKS * B_TILE_BYTES_MAX;
constexpr int P_SLOT_BYTES = STEP_BLOCKS * P_TILE_BYTES;
constexpr int GEMM_SMEM_BYTES = NB * B_SLOT_BYTES + NP * P_SLOT_BYTES +
                                1024 /*alignment slack*/ + 512 /*barriers*/;

// ---------------------------------------------------------------------------------------
// Digit matrix layout (scratch written by digitise_kernel, read by bulk copies):
// tiles of NT = nd*TOK rows x 128 contraction bytes, tile (jt, kb) at byte offset
// (jt*KB + kb) * NT*128.  Row (d*TOK + b_in) holds digit d of token jt*TOK + b_in.  Inside
// the tile, rows are 128 bytes with the 16-byte chunk index XORed with (row & 7): exactly the
// K-major 128-byte-swizzle operand layout, so a tile is one contiguous bulk copy.
// ---------------------------------------------------------------------------------------


// TPT threads per token slot b in [0, B_pad): one warp (8 tokens per block) for large batches,
// a whole block of 256 for small ones, where a row must be spread over more threads to hide
// latency.  ND digits.  A thread converts chunks of CH = 16 or 8 consecutive values; 8 when that
// spreads a row evenly over the warp (768 values = 3 x 32 chunks of 8, against 48 chunks of 16
// for 32 lanes).  `amax_bits` (optional) holds the precomputed max |value| of each token
// as float bits; otherwise the token's threads reduce it.  For int8 input (ND == 1) the
// values are their own single digit and the scale is 1.
template <typename IN_T, int ND, int TPT, int TOK, int CH>
__global__ void __launch_bounds__(256, 4)   // <= 64 registers: a batch of 4096 tokens is then one wave
digitise_kernel(const IN_T* __restrict__ in, int ld_in, int B, int B_pad, int C, int KB,
                const unsigned* __restrict__ amax_bits, int8_t* __restrict__ D, float* __restrict__ scale_out,
                int* __restrict__ zero_buf, int zero_per_token, int zero_total, int* __restrict__ status,
                unsigned long long* __restrict__ stamp, const PatchGather pg)
{
    constexpr int NT = ND * TOK;
    constexpr bool kInt = sizeof(IN_T) == 1;
    constexpr int G = CH / 4;                   // groups of four values per chunk
    constexpr int KEEP = CH == 16 ? 2 : 3;      // chunks per thread that stay in registers between the passes
    constexpr int PER_BLOCK = BLOCK_C / CH;     // chunks per 128-deep contraction block
    static_assert(TPT == 32 || TPT == 256, "one warp or one block per token");
    static_assert(CH == 16 || CH == 8, "chunk size");
    const int lane = threadIdx.x % TPT;                       // index among the token's threads
    const int b = blockIdx.x * (256 / TPT) + threadIdx.x / TPT;
    if (b >= B_pad) return;                                   // (whole block when TPT == 256)
    // launched as a programmatic dependent of the kernel before it in the stream: nothing is
    // read or written before that kernel has completed; the next kernel may be set up meanwhile
    pdl_wait();
    pdl_launch_dependents();
    tsvd_stamp_begin(stamp);
    __shared__ float red[8];
    const int jt = b / TOK, b_in = b % TOK;
    const bool live = b < B;
    const IN_T* row = in + (size_t)b * ld_in;
    const bool vec_ok = ((((uintptr_t)in) | ((size_t)ld_in * sizeof(IN_T))) & 15) == 0;
    const int n_chunks = KB * PER_BLOCK;
    // tokens that are image patches: (image, output row, output column) of this token
    int pg_n = 0, pg_ho = 0, pg_wo = 0;
    if (pg.C) {
        pg_wo = b % pg.Wo;
        pg_ho = (b / pg.Wo) % pg.Ho;
        pg_n = b / (pg.Wo * pg.Ho);
    }
    auto load_chunk = [&](int ch, float (&v)[CH]) {
        if (pg.C) {   // a chunk lies inside one run of channels (or past the row's end, or outside the image: zeros)
            const IN_T* p = ch * CH < pg.feat ? tsvd_patch_ptr<IN_T>(pg, in, pg_n, pg_ho, pg_wo, ch * CH) : nullptr;
            if (p) {
                if constexpr (CH == 16) load16<IN_T>(p, 0, CH, true, v);
                else load8<IN_T>(p, 0, CH, true, v);
            } else {
#pragma unroll
                for (int e = 0; e < CH; ++e) v[e] = 0.f;
            }
            return;
        }
        if constexpr (CH == 16) load16<IN_T>(row, ch * CH, C, vec_ok, v);
        else load8<IN_T>(row, ch * CH, C, vec_ok, v);
    };

    if (zero_buf)   // clear this token's slice of the accumulators a later kernel adds into
        for (int i = lane; i < zero_per_token; i += TPT)
            if ((size_t)b * zero_per_token + i < (size_t)zero_total) zero_buf[(size_t)b * zero_per_token + i] = 0;

    // Rows of up to KEEP chunks per thread are loaded once and kept in registers for both passes.
    const bool cached = n_chunks <= KEEP * TPT;
    float keep[KEEP][CH];
    float qscale = 1.f;
    if constexpr (!kInt) {
        float amax = 0.f;
        if (live) {
            if (amax_bits) {
                amax = __uint_as_float(amax_bits[b]);
            } else if (cached) {
#pragma unroll
                for (int j = 0; j < KEEP; ++j) {
                    const int ch = lane + j * TPT;
                    if (ch < n_chunks) {
                        load_chunk(ch, keep[j]);
#pragma unroll
                        for (int e = 0; e < CH; ++e) amax = fmaxf(amax, fabsf(keep[j][e]));
                    }
                }
            } else {
                for (int ch = lane; ch < n_chunks; ch += TPT) {
                    float v[CH];
                    load_chunk(ch, v);
#pragma unroll
                    for (int e = 0; e < CH; ++e) amax = fmaxf(amax, fabsf(v[e]));
                }
            }
            // warp-wide maximum (live is uniform across the warp)
            for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        }
        if constexpr (TPT == 256) {   // block-wide maximum (every thread of the block is here)
            if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
            __syncthreads();
#pragma unroll
            for (int w = 0; w < 8; ++w) amax = fmaxf(amax, red[w]);
        }
        // |v| <= amax < 2^E; quantise to q = rint(v * 2^(8ND-2-E)), so |q| <= 2^(8ND-2)
        const int E = tsvd_quant_exponent(amax);
        qscale = tsvd_pow2(8 * ND - 2 - E);
        if (lane == 0) scale_out[b] = tsvd_pow2(E - (8 * ND - 2));   // value = q * scale
    } else {
        if (lane == 0) scale_out[b] = 1.f;
    }

    static_assert(TOK % 8 == 0, "digit rows of one token must share their swizzle term");
    const int sw = b_in & 7;
    unsigned range_cnt = 0;   // range diagnostic: the first value of every chunk is sampled
    int8_t* tok_base = D + (size_t)jt * KB * (size_t)(NT * 128) + b_in * 128;
    // one chunk: values -> digits -> the chunk's place in the swizzled tile (zeros for a dead token)
    auto convert = [&](int ch, const float (&v)[CH]) {
        uint32_t dig[ND][G];
#pragma unroll
        for (int d = 0; d < ND; ++d)
#pragma unroll
            for (int w = 0; w < G; ++w) dig[d][w] = 0;
        if (live) {
            int q[CH];
            if constexpr (!kInt) tsvd_range_sample(range_cnt, v[0], qscale);
            if constexpr (ND <= 3) {   // |q| <= 2^22: round by adding a constant, whose image the digit offset absorbs
#pragma unroll
                for (int e = 0; e < CH; ++e) q[e] = tsvd_round_bits(v[e], qscale);
                digits_of<ND, G>(q, dig, TSVD_ROUND_BIAS);
            } else {
#pragma unroll
                for (int e = 0; e < CH; ++e) q[e] = __float2int_rn(v[e] * qscale);
                digits_of<ND, G>(q, dig);
            }
        }
        const int kb = ch / PER_BLOCK, in_block = ch % PER_BLOCK;
        const int cc = in_block * CH / 16, sub = (in_block * CH) % 16;   // 16-byte chunk of the row, offset inside it
        // (TOK is a multiple of 8, so all digit rows of a token share the swizzle term b_in & 7)
        int8_t* dst0 = tok_base + (size_t)kb * (size_t)(NT * 128) + ((cc ^ sw) << 4) + sub;
#pragma unroll
        for (int d = 0; d < ND; ++d) {
            int8_t* dst = dst0 + d * (TOK * 128);
            if constexpr (CH == 16) *reinterpret_cast<uint4*>(dst) = make_uint4(dig[d][0], dig[d][1], dig[d][2], dig[d][3]);
            else *reinterpret_cast<uint2*>(dst) = make_uint2(dig[d][0], dig[d][1]);
        }
    };
    if (cached) {
#pragma unroll
        for (int j = 0; j < KEEP; ++j) {
            const int ch = lane + j * TPT;
            if (ch < n_chunks) {
                if (!kInt && live && !amax_bits) {
                    convert(ch, keep[j]);
                } else {
                    float v[CH];
#pragma unroll
                    for (int e = 0; e < CH; ++e) v[e] = 0.f;
                    if (live) load_chunk(ch, v);
                    convert(ch, v);
                }
            }
        }
    } else {
        for (int ch = lane; ch < n_chunks; ch += TPT) {
            float v[CH];
#pragma unroll
            for (int e = 0; e < CH; ++e) v[e] = 0.f;
            if (live) load_chunk(ch, v);
            convert(ch, v);
        }
    }
    if constexpr (!kInt) {
        if (tsvd_range_flagged(range_cnt) && (threadIdx.x & 31) == 0) atomicOr(status, TSVD_DEV_RANGE);
    }
    tsvd_stamp_end(stamp);
}

// The same conversion for rows of at most 4096 padded values, 16-byte aligned and a multiple of 16
// long, as a grid that stays resident: a block of 256 threads (a chunk of 16 values per thread) walks
// over tokens blockIdx.x, blockIdx.x + gridDim.x, ... and holds the next token's chunk in registers,
// still in the input type, while it reduces, converts and stores the current one, so that a token's
// trip to memory is hidden behind the token before it.  Same digits, scales, cleared words and range
// flag as digitise_kernel.
template <typename IN_T>
struct RawChunk16 { uint4 u[sizeof(IN_T)]; };   // 16 values of 1, 2 or 4 bytes

template <typename IN_T>
__device__ __forceinline__ void raw_zero(RawChunk16<IN_T>& r)
{
#pragma unroll
    for (int i = 0; i < (int)sizeof(IN_T); ++i) r.u[i] = make_uint4(0u, 0u, 0u, 0u);
}
template <typename IN_T>
__device__ __forceinline__ void raw_load(const IN_T* __restrict__ p, RawChunk16<IN_T>& r)
{
    const uint4* p4 = reinterpret_cast<const uint4*>(p);
#pragma unroll
    for (int i = 0; i < (int)sizeof(IN_T); ++i) r.u[i] = __ldg(p4 + i);
}
template <typename IN_T>
__device__ __forceinline__ void raw_unpack(const RawChunk16<IN_T>& r, float (&v)[16])
{
    if constexpr (sizeof(IN_T) == 4) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[4 * i] = __uint_as_float(r.u[i].x); v[4 * i + 1] = __uint_as_float(r.u[i].y);
            v[4 * i + 2] = __uint_as_float(r.u[i].z); v[4 * i + 3] = __uint_as_float(r.u[i].w);
        }
    } else if constexpr (sizeof(IN_T) == 2) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const uint32_t w[4] = {r.u[i].x, r.u[i].y, r.u[i].z, r.u[i].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {   // bf16 -> fp32 is a 16-bit shift
                v[8 * i + 2 * j] = __uint_as_float(w[j] << 16);
                v[8 * i + 2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
            }
        }
    } else {
        const uint32_t w[4] = {r.u[0].x, r.u[0].y, r.u[0].z, r.u[0].w};
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = (float)(int)(int8_t)((w[j >> 2] >> (8 * (j & 3))) & 0xFF);
    }
}

template <typename IN_T, int ND, int TOK>
__global__ void __launch_bounds__(256, 4)
digitise_stream_kernel(const IN_T* __restrict__ in, int ld_in, int B, int B_pad, int C, int KB,
                       int8_t* __restrict__ D, float* __restrict__ scale_out, int* __restrict__ zero_buf,
                       int zero_per_token, int zero_total, int* __restrict__ status,
                       unsigned long long* __restrict__ stamp, const PatchGather pg)
{
    constexpr int NT = ND * TOK;
    constexpr bool kInt = sizeof(IN_T) == 1;
    static_assert(TOK % 8 == 0, "digit rows of one token must share their swizzle term");
    pdl_wait();                 // nothing is read or written before the kernel ahead has completed
    pdl_launch_dependents();
    tsvd_stamp_begin(stamp);
    __shared__ float red[2][8];
    const int ch = threadIdx.x;                   // this thread's chunk of every row
    const bool has = ch < KB * (BLOCK_C / 16);    // ... lies in the padded row
    const bool inside = ch * 16 < C;              // ... and holds values (C is a multiple of 16)
    const int kb = ch >> 3, cc = ch & 7;          // contraction block, 16-byte chunk of its 128-byte row
    const IN_T* col = in + ch * 16;
    // where this thread's chunk of token t lies (null: nothing to load): a row of a matrix, or a run of
    // channels of an image patch
    auto chunk_of = [&](int t) -> const IN_T* {
        if (t >= B || !inside) return nullptr;
        if (pg.C) return tsvd_patch_ptr<IN_T>(pg, in, t / (pg.Wo * pg.Ho), (t / pg.Wo) % pg.Ho, t % pg.Wo, ch * 16);
        return col + (size_t)t * ld_in;
    };
    RawChunk16<IN_T> nxt;
    raw_zero(nxt);
    int b = blockIdx.x;
    if (const IN_T* p0 = chunk_of(b)) raw_load(p0, nxt);
    for (int par = 0; b < B_pad; b += gridDim.x, par ^= 1) {
        const RawChunk16<IN_T> cur = nxt;
        const int bn = b + gridDim.x;
        raw_zero(nxt);
        if (const IN_T* pn = chunk_of(bn)) raw_load(pn, nxt);

        if (zero_buf)   // clear this token's slice of the accumulators a later kernel adds into
            for (int i = threadIdx.x; i < zero_per_token; i += 256)
                if ((size_t)b * zero_per_token + i < (size_t)zero_total) zero_buf[(size_t)b * zero_per_token + i] = 0;

        const bool live = b < B;
        float v[16];
        raw_unpack(cur, v);     // zeros for a dead token and outside the row
        float qscale = 1.f;
        if constexpr (!kInt) {
            float amax = 0.f;
#pragma unroll
            for (int e = 0; e < 16; ++e) amax = fmaxf(amax, fabsf(v[e]));
            for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            // the two halves of `red` alternate: a warp may write the next token's maximum while
            // another still reads this one's, never the one after (the barrier between them)
            if ((threadIdx.x & 31) == 0) red[par][threadIdx.x >> 5] = amax;
            __syncthreads();
#pragma unroll
            for (int w = 0; w < 8; ++w) amax = fmaxf(amax, red[par][w]);
            const int E = tsvd_quant_exponent(amax);
            qscale = tsvd_pow2(8 * ND - 2 - E);
            if (threadIdx.x == 0) scale_out[b] = tsvd_pow2(E - (8 * ND - 2));   // value = q * scale
        } else {
            if (threadIdx.x == 0) scale_out[b] = 1.f;
        }

        unsigned range_cnt = 0;
        if (has) {
            uint32_t dig[ND][4];
#pragma unroll
            for (int d = 0; d < ND; ++d)
#pragma unroll
                for (int w = 0; w < 4; ++w) dig[d][w] = 0;
            if (live) {
                int q[16];
                if constexpr (!kInt) tsvd_range_sample(range_cnt, v[0], qscale);
                if constexpr (ND <= 3) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) q[e] = tsvd_round_bits(v[e], qscale);
                    digits_of<ND, 4>(q, dig, TSVD_ROUND_BIAS);
                } else {
#pragma unroll
                    for (int e = 0; e < 16; ++e) q[e] = __float2int_rn(v[e] * qscale);
                    digits_of<ND, 4>(q, dig);
                }
            }
            const int jt = b / TOK, b_in = b % TOK;
            int8_t* dst = D + ((size_t)jt * KB + kb) * (size_t)(NT * 128) + b_in * 128 + ((cc ^ (b_in & 7)) << 4);
#pragma unroll
            for (int d = 0; d < ND; ++d)
                *reinterpret_cast<uint4*>(dst + d * (TOK * 128)) = make_uint4(dig[d][0], dig[d][1], dig[d][2], dig[d][3]);
        }
        if constexpr (!kInt) {
            if (tsvd_range_flagged(range_cnt) && (threadIdx.x & 31) == 0) atomicOr(status, TSVD_DEV_RANGE);
        }
    }
    tsvd_stamp_end(stamp);
}

// ---------------------------------------------------------------------------------------
// The contraction kernel (persistent: one CTA per SM walks over the tiles).  Tile (rt, jt) is
// the 128 x (ND*TOK) integer block
//   acc[r, d*TOK + i] = sum_c T[rt*128 + r, c] * digit_d(token jt*TOK + i)[c]
// accumulated in one of two tensor-memory buffers, so that the epilogue warps (combine the
// digits, apply the stage's scaling, store) work on one tile while the next is contracted.
// ---------------------------------------------------------------------------------------
enum { EPI_V = 0, EPI_U_F32 = 1, EPI_U_BF16 = 2, EPI_ACC = 3 };
enum { TAIL_T = 1, TAIL_Y = 2 };

struct GemmParams {
    const uint4* units;   // packed ternary operand
    int KB;               // contraction blocks of 128
    int R;                // logical rows (z_out / y guard)
    const int8_t* D;      // digit tiles
    const float* scale;   // per token: value = integer * scale
    int B;                // logical tokens
    const float* S;       // EPI_V: S padded to R_pad
    float* t;             // EPI_V: out [B][t_ld]
    int t_ld;
    void* z_out;          // EPI_V: optional [B][z_ld]: int32 when z_int, else fp32
    int z_ld;
    int z_int;
    void* y;              // EPI_U_*: out [B][ldy]
    int ldy;
    const float* bias;    // EPI_U_* / TAIL_Y: optional, padded to R_pad: added before the output rounding
    int* status;          // device error word
    int row_tiles;        // tiles of 128 rows
    int j_tiles;          // tiles of TOK tokens
    int ksplit;           // the contraction is cut into this many parts, one tile each (EPI_ACC when > 1)
    int* acc;             // EPI_ACC: int32 digit sums [B][ND][acc_ld], added to atomically
    int acc_ld;
    int* tile_done;       // EPI_ACC: per output tile, how many contraction parts have added their sums
    int tail;             // EPI_ACC: what the last part to finish does with the complete sums:
                          //   TAIL_T: t = S*z*scale -> p.t (+ z_out, per-token max |t| -> p.tmax)
                          //   TAIL_Y: y = sums*scale -> p.y (bf16 when p.y_bf16)
    unsigned* tmax;       // TAIL_T: per-token max |t| as float bits
    int y_bf16;
    int nb;               // depth of the digit-tile ring in steps: NB, or (resident) a whole number of panels
    int resident;         // the digit tiles of a token tile stay in shared memory across row tiles
    unsigned long long* stamp;   // time stamps of this launch, or null
    int wait_limit;       // bound of every barrier wait in units of 2^20 clocks (0: default, ~2 s)
    int test_stall;       // test hook: the digit tiles are never copied, so the waits must give up
};

// Tile index -> (row tile, token tile, contraction part); parts of one output tile are adjacent
// so that they run at the same time.
struct TileCoord { int rt, jt, kb0, kb1; };
__device__ __forceinline__ TileCoord tile_coord(const GemmParams& p, int tile)
{
    TileCoord c;
    int rest = tile;
    c.kb0 = 0;
    c.kb1 = p.KB;
    if (p.ksplit > 1) {
        const int ks = tile % p.ksplit;
        rest = tile / p.ksplit;
        c.kb0 = ks * p.KB / p.ksplit;          // ksplit <= 16 and KB < 2^20: no overflow
        c.kb1 = (ks + 1) * p.KB / p.ksplit;
    }
    c.rt = rest % p.row_tiles;
    c.jt = rest / p.row_tiles;
    return c;
}
// Each CTA takes a run of consecutive tiles (row tile fastest), so that its tiles share their
// token tile for as long as possible; the runs differ in length by at most one.
__device__ __forceinline__ void tile_range(int n_tiles, int& t0, int& t1)
{
    const int q = n_tiles / (int)gridDim.x, rem = n_tiles % (int)gridDim.x, c = (int)blockIdx.x;
    t0 = c * q + min(c, rem);
    t1 = t0 + q + (c < rem ? 1 : 0);
}
// The contraction range alone (no divisions when the contraction is not split).
__device__ __forceinline__ void tile_kb_range(const GemmParams& p, int tile, int& kb0, int& kb1)
{
    kb0 = 0;
    kb1 = p.KB;
    if (p.ksplit > 1) {
        const int ks = tile % p.ksplit;
        kb0 = ks * p.KB / p.ksplit;
        kb1 = (ks + 1) * p.KB / p.ksplit;
    }
}

template <int ND, int EPI, int TOK, int EPI_WARPS>
__global__ void __launch_bounds__(gemm_threads(EPI_WARPS), 1)
ternary_mma_kernel(const GemmParams p)
{
    constexpr int EPI_SHARES = EPI_WARPS / 4;
    constexpr int NT = ND * TOK;
    // Tiles of up to 192 columns have two accumulator buffers, so that a tile is drained while the next
    // is contracted.  WIDE: one buffer of 256 columns, for launches in which no CTA has a second tile
    // anyway; the digit ring then holds three steps of 64 KiB in the same 192 KiB.
    constexpr bool WIDE = NT > NT_MAX;
    static_assert(NT % 16 == 0 && NT <= 256 && TOK % 16 == 0, "tile shape");
    static_assert(!WIDE || EPI != EPI_ACC, "wide tiles: whole contractions only");
    constexpr uint32_t N_ACC = WIDE ? 1 : 2;
    constexpr uint32_t ACC_COLS = WIDE ? 256 : NT_MAX;
    constexpr uint32_t A_COL0 = N_ACC * ACC_COLS;
    constexpr uint32_t B_SLOT_BYTES = STEP_BLOCKS * (WIDE ? 256 : NT_MAX) * BLOCK_C;
    static_assert(A_COL0 + NA * A_SLOT_COLS <= TMEM_COLS, "tensor memory budget");
    static_assert((WIDE ? 3 : NB) * B_SLOT_BYTES <= NB * ::B_SLOT_BYTES, "digit ring inside its share of shared memory");
    constexpr uint32_t B_TILE_BYTES = NT * BLOCK_C;
    constexpr uint32_t IDESC = umma_idesc_s8(BLOCK_R, NT);

    // The contraction advances in steps of STEP_BLOCKS blocks of 128: the barrier handshakes of a
    // step cost the issuing warp about as long as four MMAs take to run, so one set of handshakes
    // has to cover more MMA time than that.
    // Three rings, because their contents live for different times:
    //   P: packed codes (4 KiB per block, shared memory), copied far ahead, freed once the
    //      expanders have read them
    //   A: expanded int8 operand (tensor memory), lives from expansion to the end of its MMAs;
    //      it never touches shared memory, whose bandwidth the digit tiles need
    //   B: digit tiles (24 KiB per block, shared memory), live from the copy's issue to the end
    //      of their MMAs
    // Step `it` uses barrier pair it % nb: "operands ready" (the digit copy's byte count plus
    // one arrival per expander warp) and "MMAs done", so that the warp that issues the MMAs
    // does one wait and one commit per step; its instruction stream is the critical path of
    // the kernel.  The digit tiles sit in slot it % nb, the expanded operand in tensor-memory
    // slot it % NA, which is free again once step it - NA is done.
    // An SM takes in about 64 bytes per clock from L2, and a block's 24 KiB digit tile plus
    // 4 KiB of codes at that rate take longer than its four MMAs.  So when the whole contraction
    // fits the ring the ring depth nb is a whole number of panels (all steps of a tile), a CTA
    // walks consecutive row tiles of one token tile, and the digit tiles are copied only when the
    // token tile changes: per block only the 4 KiB of codes then come from L2.
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* b_tiles = smem;                                 // NB x 48 KiB, 1024-aligned
    uint8_t* p_tiles = b_tiles + NB * ::B_SLOT_BYTES;        // NP x 8 KiB
    uint64_t* bars = reinterpret_cast<uint64_t*>(p_tiles + NP * P_SLOT_BYTES);
    uint64_t* pfull_bar = bars;                      // [NP] packed codes landed
    uint64_t* pempty_bar = pfull_bar + NP;           // [NP] expanders have read them
    uint64_t* ready_bar = pempty_bar + NP;           // [NB] digit tile landed and expanded operand written
    uint64_t* done_bar = ready_bar + NB;             // [NB][STEP_BLOCKS] the MMAs of block j of the step have completed
    uint64_t* accfull_bar = done_bar + NB * STEP_BLOCKS;   // [2] all MMAs of a tile have completed
    uint64_t* accempty_bar = accfull_bar + 2;        // [2] the epilogue has drained the accumulator
    uint64_t* tail_bar = accempty_bar + 2;           // [2] split contraction: epilogue warps meet, outcome is in
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail_bar + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);   // [2]: flag, wait limit
    volatile int* tail_last = abort_flag + 2;        // whether this CTA finished its output tile last

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = p.KB;
    const int n_tiles = p.row_tiles * p.j_tiles * p.ksplit;
    // Tile L of this CTA.  Resident digit tiles: a run of consecutive tiles (they share the token
    // tile).  Otherwise strided, so that the CTAs running at one time read the same digit tiles
    // and those stay hot in L2.
    int tile_first = (int)blockIdx.x, tile_step = (int)gridDim.x;
    int tile_count = (n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    if (p.resident) {
        int t0, t1;
        tile_range(n_tiles, t0, t1);
        tile_first = t0;
        tile_step = 1;
        tile_count = t1 - t0;
    }
    const uint32_t nb = (uint32_t)p.nb;

    if (threadIdx.x == 0) {
        for (int s = 0; s < NP; ++s) { mbar_init(&pfull_bar[s], 1); mbar_init(&pempty_bar[s], 4); }
        for (int s = 0; s < NB; ++s) {
            mbar_init(&ready_bar[s], 5);   // the copy's expect-tx arrival + one per expander warp of the group
            for (int j = 0; j < STEP_BLOCKS; ++j) mbar_init(&done_bar[s * STEP_BLOCKS + j], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&accfull_bar[i], 1);
            mbar_init(&accempty_bar[i], EPI_WARPS);  // one arrival per epilogue warp
        }
        mbar_init(&tail_bar[0], EPI_WARPS);
        mbar_init(&tail_bar[1], 1);
        abort_flag[0] = 0;
        abort_flag[1] = p.wait_limit > 0 ? p.wait_limit : kWaitLimitDefault;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Launched as a programmatic dependent of the kernel before it in the stream (the one that
    // wrote the digits): everything up to here, and the copies of the packed codes (which no
    // kernel writes), may overlap with that kernel; all other warps wait for it to complete.
    if (warp != 2) pdl_wait();
    pdl_launch_dependents();
    tsvd_stamp_begin(p.stamp);

    // Waiting for parity 1 on a barrier that has not completed a phase yet returns at once,
    // which is what a consumer-release barrier needs on its first use.
    if (warp == 0 || warp == 2) {
        // ---- copy producers: warp 0 streams the digit tiles, warp 2 the packed codes.  The whole
        //      warp runs the loop (uniform control flow); one elected lane issues the copies ----
        {
            const bool is_b = warp == 0;
            const uint32_t depth = is_b ? nb : (uint32_t)NP;
            const int panels = p.nb / ((KB + STEP_BLOCKS - 1) / STEP_BLOCKS);   // resident: token panels the ring holds
            uint64_t* full = is_b ? ready_bar : pfull_bar;
            // a digit slot is free when the last block of the step that used it is done
            uint64_t* empty = is_b ? done_bar + (STEP_BLOCKS - 1) : pempty_bar;
            const uint32_t empty_stride = is_b ? (uint32_t)STEP_BLOCKS : 1u;
            // the blocks of a step are adjacent both in global memory and in the slot
            const uint32_t blk_bytes = is_b ? B_TILE_BYTES : (uint32_t)P_TILE_BYTES;
            const uint32_t slot_bytes = is_b ? (uint32_t)B_SLOT_BYTES : (uint32_t)P_SLOT_BYTES;
            uint8_t* ring = is_b ? b_tiles : p_tiles;
            uint32_t slot = 0, phase = 0, issued = 0;
            bool alive = true;
            for (int L = 0, tile = tile_first; L < tile_count && alive; ++L, tile += tile_step) {
                const TileCoord tc = tile_coord(p, tile);
                const uint8_t* src = is_b ? reinterpret_cast<const uint8_t*>(p.D) + (size_t)tc.jt * KB * B_TILE_BYTES
                                          : reinterpret_cast<const uint8_t*>(p.units) + (size_t)tc.rt * KB * P_TILE_BYTES;
                // Resident digit tiles: the ring holds whole panels (all steps of a token tile),
                // tile L of this CTA uses panel L % panels, and if the tile that used it before had
                // the same token tile the data are there already: only the barrier is armed.
                bool copy = true;
                if (is_b && p.resident) copy = L < panels || (tile - panels) / p.row_tiles != tc.jt;
                for (int kb = tc.kb0; kb < tc.kb1; kb += STEP_BLOCKS, ++issued) {
                    const uint32_t bytes = (uint32_t)min(STEP_BLOCKS, tc.kb1 - kb) * blk_bytes;
                    if (!mbar_wait(&empty[slot * empty_stride], phase ^ 1, abort_flag)) { alive = false; break; }
                    if (is_b && p.test_stall) { alive = false; break; }   // nothing will ever land
                    TSVD_BOUND(p.status, slot < depth && bytes <= slot_bytes && kb + (int)(bytes / blk_bytes) <= KB &&
                                             tc.rt < p.row_tiles && tc.jt < p.j_tiles);
                    if (elect_one()) {
                        if (copy) {
                            mbar_arrive_expect_tx(&full[slot], bytes);
                            bulk_g2s(ring + slot * slot_bytes, src + (size_t)kb * blk_bytes, bytes, &full[slot]);
                        } else {
                            mbar_arrive(&full[slot]);
                        }
                    }
                    __syncwarp();
                    if (++slot == depth) { slot = 0; phase ^= 1; }
                }
            }
            if (*abort_flag && lane == 0) {
                // a wait gave up somewhere: let this CTA's own copies land before it exits (bounded)
                const uint32_t first = issued > depth ? issued - depth : 0u;
                for (uint32_t j = first; j < issued; ++j) {
                    uint64_t* bar = &full[j % depth];
                    const uint32_t ph = (j / depth) & 1;
                    for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(bar, ph); ++spin) {}
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issue.  The whole warp runs the loop so that slot, phase and the operand
        //      descriptors stay warp-uniform (the MMA instructions take them from the uniform
        //      register file); one elected lane issues the MMAs and commits. ----
        {
            uint32_t slot = 0, phase = 0, aslot = 0;
            const uint64_t b_desc0 = umma_desc_k_sw128(smem_u32(b_tiles));
            // readiness of the next slot is tested (without blocking) while the current step's
            // MMAs are being issued, so that the barrier's latency is off the issue path
            bool ready = mbar_test_wait(&ready_bar[0], 0);
            bool alive = true;
            for (int L = 0, tile = tile_first; L < tile_count && alive; ++L, tile += tile_step) {
                const uint32_t buf = (uint32_t)L % N_ACC;
                if (!mbar_wait(&accempty_bar[buf], (((uint32_t)L / N_ACC) & 1) ^ 1, abort_flag)) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * (uint32_t)ACC_COLS;
                int kb0, kb1;
                tile_kb_range(p, tile, kb0, kb1);
                for (int kb = kb0; kb < kb1; kb += STEP_BLOCKS) {
                    const int nblk = min(STEP_BLOCKS, kb1 - kb);
                    if (!ready && !mbar_wait(&ready_bar[slot], phase, abort_flag)) { alive = false; break; }
                    tc_fence_after_sync();
                    const uint32_t a_tmem = tmem_base + (uint32_t)A_COL0 + aslot * (uint32_t)A_SLOT_COLS;
                    const uint64_t b_desc = b_desc0 + (uint64_t)(slot * (B_SLOT_BYTES >> 4));
                    TSVD_BOUND(p.status, slot < nb && aslot < (uint32_t)NA && nblk >= 1 && nblk <= STEP_BLOCKS);
                    const uint32_t cur = slot;
                    if (++slot == nb) { slot = 0; phase ^= 1; }
                    aslot = (aslot + 1) & (NA - 1);
                    if (elect_one()) {
                        // 32 contraction elements per instruction: 8 columns of A, 32 bytes of
                        // the swizzled 128-byte rows of B
#pragma unroll
                        for (int j = 0; j < STEP_BLOCKS; ++j) {
                            if (j < nblk) {
#pragma unroll
                                for (int k = 0; k < BLOCK_C / UMMA_K; ++k)
                                    umma_s8_ts(d_tmem, a_tmem + (uint32_t)(j * A_BLOCK_COLS + k * (UMMA_K / 4)),
                                               b_desc + (uint64_t)(j * (B_TILE_BYTES >> 4) + k * (UMMA_K >> 4)), IDESC,
                                               kb != kb0 || j != 0 || k != 0);
                            }
                            // block j of the step is done (a block the step does not have counts as
                            // done too): its part of the A slot is free NA steps on, and after the
                            // last block the digit slot
                            umma_commit(&done_bar[cur * STEP_BLOCKS + j]);
                        }
                    }
                    __syncwarp();
                    ready = mbar_test_wait(&ready_bar[slot], phase);
                }
                if (elect_one()) umma_commit(&accfull_bar[buf]);
                __syncwarp();
            }
        }
    } else if (warp >= EXP_WARP0 && warp < EPI_WARP0) {
        // ---- expanders: thread = row of the tile = tensor-memory lane (warp w may touch lanes
        //      32*(w%4)..+31); the groups of four warps take the steps in turn, so that the
        //      barrier and memory latencies of one step overlap with work on the next ----
        const int r = (threadIdx.x - EXP_WARP0 * 32) & 127;   // 0..127
        const uint32_t group = (uint32_t)(warp - EXP_WARP0) >> 2;
        uint32_t it = 0, sb = 0, phb = 0;   // step counter; its slot and phase in the digit-tile ring
        bool alive = true;
        for (int L = 0, tile = tile_first; L < tile_count && alive; ++L, tile += tile_step) {
            int kb0, kb1;
            tile_kb_range(p, tile, kb0, kb1);
            for (int kb = kb0; kb < kb1; kb += STEP_BLOCKS, ++it, sb = (sb + 1 == nb ? 0u : sb + 1), phb ^= (sb == 0)) {
                if (it % EXP_GROUPS != group) continue;
                const int nblk = min(STEP_BLOCKS, kb1 - kb);
                const int sp = it % NP, sa = it % NA;
                TSVD_BOUND(p.status, sb < nb && r < BLOCK_R && A_COL0 + sa * A_SLOT_COLS + STEP_BLOCKS * A_BLOCK_COLS <= TMEM_COLS);
                if (!mbar_wait(&pfull_bar[sp], (it / NP) & 1, abort_flag)) { alive = false; break; }
                const uint4* packed = reinterpret_cast<const uint4*>(p_tiles + sp * P_SLOT_BYTES);
                const uint32_t a_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(A_COL0 + sa * A_SLOT_COLS);
                // expand the whole step into registers first, so that only the stores are left to do
                // once the slot is free
                uint32_t o[STEP_BLOCKS][32];   // per block: the row's 128 int8 values, four per 32-bit column
#pragma unroll
                for (int j = 0; j < STEP_BLOCKS; ++j) {
                    if (j < nblk) {
#pragma unroll
                        for (int g = 0; g < 2; ++g) {
                            const uint4 u = packed[j * 256 + g * 128 + r];
                            tsvd_expand16(u.x, *reinterpret_cast<uint32_t(*)[4]>(&o[j][g * 16 + 0]));
                            tsvd_expand16(u.y, *reinterpret_cast<uint32_t(*)[4]>(&o[j][g * 16 + 4]));
                            tsvd_expand16(u.z, *reinterpret_cast<uint32_t(*)[4]>(&o[j][g * 16 + 8]));
                            tsvd_expand16(u.w, *reinterpret_cast<uint32_t(*)[4]>(&o[j][g * 16 + 12]));
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&pempty_bar[sp]);   // all codes of the step are in registers
                bool ok = true;
#pragma unroll
                for (int j = 0; j < STEP_BLOCKS; ++j) {
                    if (j < nblk && ok) {
                        if (it >= (uint32_t)NA) {   // this part of the A slot is free once block j of step it - NA is done
                            uint32_t sd = sb + nb - NA, phd = phb ^ 1;   // its slot, NA back (nb >= NA), and phase
                            if (sd >= nb) { sd -= nb; phd = phb; }
                            ok = mbar_wait(&done_bar[sd * STEP_BLOCKS + j], phd, abort_flag);
                            tc_fence_after_sync();
                        }
                        if (ok) tmem_st32(a_addr + (uint32_t)(j * A_BLOCK_COLS), o[j]);
                    }
                }
                if (!ok) { alive = false; break; }
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ready_bar[sb]);
            }
        }
    } else if (warp >= EPI_WARP0) {
        // ---- epilogue: warp w reads tensor-memory lanes 32*(w%4) .. +31 and takes its share
        //      (all, or every second) of the tile's groups of 8 tokens ----
        const int lane_grp = warp & 3;
        const int half = (warp - EPI_WARP0) >> 2;
        const int row_in = lane_grp * 32 + lane;
        uint32_t local = 0;
        for (int tile = tile_first; local < (uint32_t)tile_count; tile += tile_step, ++local) {
            const TileCoord tc = tile_coord(p, tile);
            const int rt = tc.rt, jt = tc.jt;
            const int row = rt * BLOCK_R + row_in;
            TSVD_BOUND(p.status, rt < p.row_tiles && jt < p.j_tiles && row < p.row_tiles * BLOCK_R);
            const uint32_t buf = local % N_ACC;
            // this warp takes its share of the groups of 8 tokens
            constexpr int N_GROUPS = TOK / 8;
            constexpr int MY_GROUPS = N_GROUPS / EPI_SHARES;
            static_assert(N_GROUPS % EPI_SHARES == 0, "the epilogue warps of a lane group share the token groups evenly");
            float s_row = 0.f;   // EPI_V: S of the row; EPI_U_*: the row's bias
            if constexpr (EPI == EPI_V) s_row = p.S[row];
            if constexpr (EPI == EPI_U_F32 || EPI == EPI_U_BF16) s_row = p.bias ? __ldg(p.bias + row) : 0.f;
            const bool row_ok = row < p.R;
            if (!mbar_wait(&accfull_bar[buf], (local / N_ACC) & 1, abort_flag)) break;
            tc_fence_after_sync();
            const uint32_t t_lane = tmem_base + buf * (uint32_t)ACC_COLS + ((uint32_t)(lane_grp * 32) << 16);
#pragma unroll
            for (int k = 0; k < MY_GROUPS; ++k) {
                const int g = half + EPI_SHARES * k;
                uint32_t acc[ND][8];
#pragma unroll
                for (int d = 0; d < ND; ++d) tmem_ld8(t_lane + (uint32_t)(d * TOK + g * 8), acc[d]);
                const int b0 = jt * TOK + g * 8;
                // the group's eight per-token scales: every lane reads the same 32 bytes (the
                // array is padded to whole tiles), while the tensor-memory loads are in flight
                float sc[8];
                if constexpr (EPI != EPI_ACC) {
                    const float4 s0 = __ldg(reinterpret_cast<const float4*>(p.scale + b0));
                    const float4 s1 = __ldg(reinterpret_cast<const float4*>(p.scale + b0 + 4));
                    sc[0] = s0.x; sc[1] = s0.y; sc[2] = s0.z; sc[3] = s0.w;
                    sc[4] = s1.x; sc[5] = s1.y; sc[6] = s1.z; sc[7] = s1.w;
                }
                tmem_ld_wait();
                const int n_live = min(8, p.B - b0);   // uniform across the warp
                // whole group inside the batch and every row of the warp inside the matrix: no guards
                const bool full = n_live == 8 && __all_sync(0xffffffffu, row_ok);
                if constexpr (EPI == EPI_ACC) {
                    // part of a split contraction: add the raw digit sums to the global accumulators
                    // (integer adds commute exactly, so the result does not depend on arrival order)
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        if (i < n_live) {
#pragma unroll
                            for (int d = 0; d < ND; ++d)
                                atomicAdd(p.acc + ((size_t)(b0 + i) * ND + d) * p.acc_ld + row, (int)acc[d][i]);
                        }
                    }
                } else {
                // digits -> fp32: lo and hi are exact 32-bit integers; their conversions and the
                // fused multiply-add round at 2^-24 of |hi|*65536 and |lo|.  (64-bit integer and
                // double conversions are far too slow on this part to sit in this loop.)
                float val[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    float f;
                    if constexpr (ND == 1) {
                        f = (float)(int)acc[0][i];
                    } else if constexpr (ND == 2) {
                        f = (float)((int)acc[0][i] + ((int)acc[1][i] << 8));
                    } else {
                        const int lo = (int)acc[0][i] + ((int)acc[1][i] << 8);
                        int hi = (int)acc[2][i];
                        if constexpr (ND == 4) hi += (int)acc[3][i] << 8;
                        f = fmaf((float)hi, 65536.f, (float)lo);
                    }
                    val[i] = f * sc[i];   // a power of two: exact
                    if constexpr (EPI == EPI_U_F32 || EPI == EPI_U_BF16) val[i] += s_row;   // bias (0 without one)
                }
                if constexpr (EPI == EPI_V) {
                    float* tp = p.t + (size_t)b0 * p.t_ld + row;
                    if (n_live == 8) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) tp[(size_t)i * p.t_ld] = s_row * val[i];   // the K multiplications (Table S1)
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            if (i < n_live) tp[(size_t)i * p.t_ld] = s_row * val[i];
                    }
                    if (p.z_out && row_ok) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            if (i < n_live) {
                                const size_t o = (size_t)(b0 + i) * p.z_ld + row;
                                if (p.z_int) reinterpret_cast<int*>(p.z_out)[o] = (int)acc[0][i];
                                else reinterpret_cast<float*>(p.z_out)[o] = val[i];
                            }
                        }
                    }
                } else if constexpr (EPI == EPI_U_F32) {
                    float* yp = reinterpret_cast<float*>(p.y) + (size_t)b0 * p.ldy + row;
                    if (full) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) yp[(size_t)i * p.ldy] = val[i];
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            if (row_ok && i < n_live) yp[(size_t)i * p.ldy] = val[i];
                    }
                } else {
                    __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(p.y) + (size_t)b0 * p.ldy + row;
                    if (full) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) yp[(size_t)i * p.ldy] = __float2bfloat16_rn(val[i]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            if (row_ok && i < n_live) yp[(size_t)i * p.ldy] = __float2bfloat16_rn(val[i]);
                    }
                }
                }   // EPI != EPI_ACC
            }
            // all tensor-memory reads of this buffer are done: hand it back to the MMA thread
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&accempty_bar[buf]);

            if constexpr (EPI == EPI_ACC) {
                // Split contraction: the part that finishes an output tile last turns the complete
                // sums into the stage's result.  (Sums were added with device-scope atomics; the
                // fence orders them before the counter.)
                __threadfence();
                __syncwarp();
                if (lane == 0) mbar_arrive(&tail_bar[0]);
                if (!mbar_wait(&tail_bar[0], local & 1, abort_flag)) break;
                if (warp == EPI_WARP0 && lane == 0) {
                    const int out_tile = jt * p.row_tiles + rt;
                    *tail_last = atomicAdd(p.tile_done + out_tile, 1) == p.ksplit - 1;
                    __threadfence();
                    mbar_arrive(&tail_bar[1]);
                }
                if (!mbar_wait(&tail_bar[1], local & 1, abort_flag)) break;
                if (*tail_last) {
                  // this warp: rows 32*(warp%4).. and its share of the tile's groups of 8 tokens
#pragma unroll 1
                  for (int tg = half; tg < TOK / 8; tg += EPI_SHARES) {
                    const int b0 = jt * TOK + tg * 8;
                    const bool row_ok = row < p.R;
                    const float s_row = p.tail == TAIL_T ? p.S[row] : (p.bias ? __ldg(p.bias + row) : 0.f);
                    // all loads first (they are independent and come from L2), then the arithmetic
                    int a[8][ND];
                    float sc[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const bool live = b0 + i < p.B;              // uniform across the warp
                        sc[i] = live ? __ldg(p.scale + b0 + i) : 0.f;
#pragma unroll
                        for (int d = 0; d < ND; ++d)
                            a[i][d] = live ? __ldcg(p.acc + ((size_t)(b0 + i) * ND + d) * p.acc_ld + row) : 0;
                    }
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int b = b0 + i;
                        if (b >= p.B) break;                         // uniform across the warp
                        float f;
                        if constexpr (ND == 1) f = (float)a[i][0];
                        else if constexpr (ND == 2) f = (float)(a[i][0] + (a[i][1] << 8));
                        else {
                            const int lo = a[i][0] + (a[i][1] << 8);
                            int hi = a[i][2];
                            if constexpr (ND == 4) hi += a[i][3] << 8;
                            f = fmaf((float)hi, 65536.f, (float)lo);
                        }
                        const float val = f * sc[i];
                        if (p.tail == TAIL_T) {
                            const float tv = s_row * val;             // the K multiplications (Table S1)
                            p.t[(size_t)b * p.t_ld + row] = tv;
                            if (p.z_out && row_ok) {
                                if (p.z_int) reinterpret_cast<int*>(p.z_out)[(size_t)b * p.z_ld + row] = a[i][0];
                                else reinterpret_cast<float*>(p.z_out)[(size_t)b * p.z_ld + row] = val;
                            }
                            const unsigned m = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(tv)));
                            if (lane == 0) atomicMax(p.tmax + b, m);
                        } else if (row_ok) {
                            const float yv = val + s_row;   // bias (0 without one)
                            if (p.y_bf16)
                                reinterpret_cast<__nv_bfloat16*>(p.y)[(size_t)b * p.ldy + row] = __float2bfloat16_rn(yv);
                            else
                                reinterpret_cast<float*>(p.y)[(size_t)b * p.ldy + row] = yv;
                        }
                    }
                  }
                }
            }
        }
    }

    // ---- teardown ----
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) atomicOr(p.status, TSVD_DEV_TIMEOUT);
    if (threadIdx.x == 0) tsvd_stamp_end(p.stamp);
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

template <typename IN_T, int ND, int TOK = tokens_per_tile(ND)>
cudaError_t launch_digitise(const IN_T* in, int ld_in, int B, int C, int KB, const unsigned* amax_bits,
                            int8_t* D, float* scale, int* zero_buf, int zero_total, int* status,
                            unsigned long long* stamp, cudaStream_t stream, const PatchGather* gather = nullptr)
{
    const PatchGather pg = gather ? *gather : PatchGather();
    const int B_pad = (B + TOK - 1) / TOK * TOK;
    const int zero_per_token = (zero_total + B_pad - 1) / B_pad;   // every token slot clears a share
    // rows of 1024 to 4096 padded values that vector loads can read whole, without a maximum given:
    // the resident form, as many blocks as the GPU holds at one time (rows under 2048 values leave
    // half of a block's threads without a chunk: there a batch large enough for the warp-per-token
    // form below keeps that form, which measured 4% faster on a convolution's 25088 patches of 1152)
    if (!amax_bits && KB >= 8 && KB <= 32 && (KB >= 16 || B_pad * 32 < 148 * 1024) && C % 16 == 0 &&
        ((((uintptr_t)in) | ((size_t)(gather ? 16 : ld_in) * sizeof(IN_T))) & 15) == 0) {
        int dev = 0, sms = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const int resident = 4 * sms;
        PdlLaunch cfg((unsigned)(B_pad < resident ? B_pad : resident), 256, 0, stream);
        const cudaError_t e = cudaLaunchKernelEx(&cfg.cfg, digitise_stream_kernel<IN_T, ND, TOK>, in, ld_in, B, B_pad, C, KB, D,
                                                 scale, zero_buf, zero_per_token, zero_total, status, stamp, pg);
        tsvd_count_launch();
        return e != cudaSuccess ? e : cudaGetLastError();
    }
    // one warp per token when that gives enough warps to fill the GPU, or for short rows
    PdlLaunch cfg((B_pad * 32 >= 148 * 1024 || KB < 8) ? (unsigned)((B_pad + 7) / 8) : (unsigned)B_pad, 256, 0, stream);
    cudaError_t e;
    if (B_pad * 32 >= 148 * 1024 || KB < 8) {   // (same rule as above)
        // chunks of 8 values when chunks of 16 would leave part of the warp without work in the last
        // round and the row still fits the registers (three chunks of 8 per lane)
        if ((KB * 8) % 32 != 0 && KB * 16 <= 3 * 32)
            e = cudaLaunchKernelEx(&cfg.cfg, digitise_kernel<IN_T, ND, 32, TOK, 8>, in, ld_in, B, B_pad, C, KB, amax_bits, D,
                                   scale, zero_buf, zero_per_token, zero_total, status, stamp, pg);
        else
            e = cudaLaunchKernelEx(&cfg.cfg, digitise_kernel<IN_T, ND, 32, TOK, 16>, in, ld_in, B, B_pad, C, KB, amax_bits,
                                   D, scale, zero_buf, zero_per_token, zero_total, status, stamp, pg);
    } else {
        e = cudaLaunchKernelEx(&cfg.cfg, digitise_kernel<IN_T, ND, 256, TOK, 16>, in, ld_in, B, B_pad, C, KB, amax_bits, D,
                               scale, zero_buf, zero_per_token, zero_total, status, stamp, pg);
    }
    tsvd_count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

template <int ND, int EPI, int TOK, int EPIW>
cudaError_t launch_gemm_w(const GemmParams& p, int row_tiles, cudaStream_t stream)
{
    static bool attr_set[64] = {};   // per instantiation and device
    int dev = 0;
    cudaError_t e0 = cudaGetDevice(&dev);
    if (e0 != cudaSuccess) return e0;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(ternary_mma_kernel<ND, EPI, TOK, EPIW>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_BYTES);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    GemmParams q = p;
    q.row_tiles = row_tiles;
    q.j_tiles = (p.B + TOK - 1) / TOK;
    if (q.ksplit < 1) q.ksplit = 1;
    // A contraction of at most NB steps leaves room to keep a token tile's digit tiles in shared
    // memory while the CTA walks the row tiles: the ring then holds whole panels (a tile's steps).
    q.nb = NB;
    q.resident = 0;
    const int steps = (q.KB + STEP_BLOCKS - 1) / STEP_BLOCKS;
    if (ND * TOK > NT_MAX) {
        q.nb = 3;   // tiles of 256 columns: three steps of 64 KiB fill the digit ring
    } else if (q.ksplit == 1 && steps <= NB) {
        q.nb = steps * (NB / steps);
        q.resident = 1;
    }
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int n_tiles = q.row_tiles * q.j_tiles * q.ksplit;
    const int grid = n_tiles < sms ? n_tiles : sms;
    PdlLaunch cfg((unsigned)grid, (unsigned)gemm_threads(EPIW), GEMM_SMEM_BYTES, stream);
    const cudaError_t e = cudaLaunchKernelEx(&cfg.cfg, ternary_mma_kernel<ND, EPI, TOK, EPIW>, (const GemmParams)q);
    tsvd_count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

template <int ND, int EPI, int TOK = tokens_per_tile(ND)>
cudaError_t launch_gemm(const GemmParams& p, int row_tiles, cudaStream_t stream)
{
    if constexpr (EPI != EPI_ACC) {
        if (four_epilogue_warps(p.KB, TOK)) return launch_gemm_w<ND, EPI, TOK, 4>(p, row_tiles, stream);
    }
    return launch_gemm_w<ND, EPI, TOK, EPI_WARPS_MAX>(p, row_tiles, stream);
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// digit counts: int8 activations are their own single digit; bf16 needs 3 (22-bit fixed
// point holds every bf16 value within 2^-12 of the token's largest exactly); fp32 and the
// intermediate t use 4 (30 bits).
inline int digits_for_x(tsvd_dtype_t dt, bool wide) { return dt == TSVD_I8 ? 1 : (dt == TSVD_BF16 && !wide) ? 3 : 4; }
constexpr int ND_T = 4;
// Tokens per tile of the V-stage.  A tile's time hardly depends on its width (the expanders and the
// issuing warp set it), so the widest tile is the rule; int8 activations (one digit: 192 tokens a tile)
// take tiles of 128 tokens where that leaves fewer padded tokens, e.g. 256 tokens as 2 x 128 instead of
// 192 + 64 (V-stage of a 8192 x 4096 matrix at 256 tokens: 14.1 -> 12.0 us).
constexpr int TOK_I8_NARROW = 128;
// Tokens per tile of the U-stage: 48 (four digits, 192 columns, two accumulator buffers), or 64 (256
// columns, one buffer) when that brings the number of tiles down to at most one per SM, where nothing
// would overlap with a second buffer anyway (4096 rows x 256 tokens: 32 x 6 = 192 tiles in two rounds
// against 32 x 4 = 128 in one).
constexpr int TOK_T_WIDE = 64;
inline int tokens_of_four_digit_tile(int row_tiles, int B)
{
    static int sms = 0;
    if (sms == 0) {
        int dev = 0, n = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        sms = n;
    }
    const int regular = tokens_per_tile(ND_T);
    const long long tiles_regular = (long long)row_tiles * ((B + regular - 1) / regular);
    const long long tiles_wide = (long long)row_tiles * ((B + TOK_T_WIDE - 1) / TOK_T_WIDE);
    return tiles_regular > sms && tiles_wide <= sms ? TOK_T_WIDE : regular;
}
inline int tokens_of_t_tile(const tsvd_handle_s* h, int B) { return tokens_of_four_digit_tile(h->U.R_pad / BLOCK_R, B); }
// (the V-stage of four-digit activations -- fp32, or bf16 on request -- follows the same rule)
inline int tokens_of_x_tile(const tsvd_handle_s* h, int ndx, int B)
{
    if (ndx == 4) return tokens_of_four_digit_tile(h->V.R_pad / BLOCK_R, B);
    const int wide_tile = tokens_per_tile(ndx);
    if (ndx != 1) return wide_tile;
    const long long padded_wide = (B + wide_tile - 1LL) / wide_tile * wide_tile;
    const long long padded_narrow = (B + TOK_I8_NARROW - 1LL) / TOK_I8_NARROW * TOK_I8_NARROW;
    return 8 * padded_narrow <= 7 * padded_wide ? TOK_I8_NARROW : wide_tile;
}

struct TensorWs {
    int8_t* Dx; float* scale_x; float* t; unsigned* tmax; int8_t* Dt; float* scale_t;
    size_t total;
};

TensorWs carve(const tsvd_handle_s* h, int B, tsvd_dtype_t dt, bool wide, void* base)
{
    const int ndx = digits_for_x(dt, wide);
    const int tokx = tokens_of_x_tile(h, ndx, B), tokt = tokens_of_t_tile(h, B);
    const size_t Bx = align_up(B, tokx), Bt = align_up(B, tokt);
    const size_t Bmax = Bx > Bt ? Bx : Bt;
    const size_t KBv = h->V.C_pad / BLOCK_C, KBu = h->U.C_pad / BLOCK_C;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return o; };
    const size_t o_dx = take(Bx * ndx * KBv * 128);
    const size_t o_sx = take(Bmax * sizeof(float));
    const size_t o_t = take(Bmax * (size_t)h->V.R_pad * sizeof(float));
    const size_t o_tm = take(Bmax * sizeof(unsigned));
    const size_t o_dt = take(Bt * ND_T * KBu * 128);
    const size_t o_st = take(Bmax * sizeof(float));
    TensorWs w;
    char* b = reinterpret_cast<char*>(base);
    w.Dx = reinterpret_cast<int8_t*>(b + o_dx);
    w.scale_x = reinterpret_cast<float*>(b + o_sx);
    w.t = reinterpret_cast<float*>(b + o_t);
    w.tmax = reinterpret_cast<unsigned*>(b + o_tm);
    w.Dt = reinterpret_cast<int8_t*>(b + o_dt);
    w.scale_t = reinterpret_cast<float*>(b + o_st);
    w.total = off;
    return w;
}

}  // namespace

namespace {

constexpr int SMALL_TOK = 16;        // tokens per tile on the small-batch path
constexpr int SMALL_MAX_B = 512;   // (the split form also has to be preferred: few row tiles, long contractions)

struct SmallWs {
    int8_t* Dx; float* scale_x; int* zacc; float* t; int8_t* Dt; float* scale_t; int* yacc;
    int zacc_ints, yacc_ints;     // sums + per-token max + per-tile counters: cleared as one range
    size_t total;
};

SmallWs carve_small(const tsvd_handle_s* h, int B, tsvd_dtype_t dt, bool wide, void* base)
{
    const int ndx = digits_for_x(dt, wide);
    const size_t Bp = align_up(B, SMALL_TOK);
    const size_t KBv = h->V.C_pad / BLOCK_C, KBu = h->U.C_pad / BLOCK_C;
    const size_t j_tiles = Bp / SMALL_TOK;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return o; };
    SmallWs w;
    // [sums Bp*nd*R_pad][max |t| per token Bp][tile counters]
    w.zacc_ints = (int)(Bp * ndx * (size_t)h->V.R_pad + Bp + (size_t)(h->V.R_pad / BLOCK_R) * j_tiles);
    w.yacc_ints = (int)(Bp * ND_T * (size_t)h->U.R_pad + (size_t)(h->U.R_pad / BLOCK_R) * j_tiles);
    const size_t o_dx = take(Bp * ndx * KBv * 128);
    const size_t o_sx = take(Bp * sizeof(float));
    const size_t o_za = take((size_t)w.zacc_ints * sizeof(int));
    const size_t o_t = take(Bp * (size_t)h->V.R_pad * sizeof(float));
    const size_t o_dt = take(Bp * ND_T * KBu * 128);
    const size_t o_st = take(Bp * sizeof(float));
    const size_t o_ya = take((size_t)w.yacc_ints * sizeof(int));
    char* b = reinterpret_cast<char*>(base);
    w.Dx = reinterpret_cast<int8_t*>(b + o_dx);
    w.scale_x = reinterpret_cast<float*>(b + o_sx);
    w.zacc = reinterpret_cast<int*>(b + o_za);
    w.t = reinterpret_cast<float*>(b + o_t);
    w.Dt = reinterpret_cast<int8_t*>(b + o_dt);
    w.scale_t = reinterpret_cast<float*>(b + o_st);
    w.yacc = reinterpret_cast<int*>(b + o_ya);
    w.total = off;
    return w;
}

// how many parts to cut the contraction into so that the tiles about fill the GPU
int pick_ksplit(int out_tiles, int KB)
{
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    int ks = sms / (out_tiles > 0 ? out_tiles : 1);
    if (ks > KB) ks = KB;
    if (ks > 16) ks = 16;
    return ks < 1 ? 1 : ks;
}

// Whether a batch of at most SMALL_MAX_B tokens runs the split-contraction form below rather than the tile
// kernels (one tile of tokens per row tile).  Both are bound by the blocks of 128 columns a CTA walks through
// (about 0.2 us each): per stage the tile kernels take rounds x KB of them, the split form rounds x KB / parts,
// but its integer atomics, last-arriver tails and heavier launches cost about 8 us more per forward (40 blocks).
// Measured (bf16, 20 to 48 tokens, us, split / tiles): 4096^3 38 / 29, 768^3 24 / 16, 2048 x 8192 x 2048 28 / 31,
// 1024 x 16384 x 1024 28 / 43, 256 x 32768 x 256 27 / 70, 128 x 16384 x 16384 92 / 77: the rule reproduces each.
bool prefer_split_form(const tsvd_handle_s* h, int B)
{
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int j16 = (B + SMALL_TOK - 1) / SMALL_TOK;
    long long tiles_cost = 0, split_cost = 40;
    for (const PackedMat* m : {&h->V, &h->U}) {
        const int rows = m->R_pad / BLOCK_R, KB = m->C_pad / BLOCK_C;
        tiles_cost += (long long)((rows + sms - 1) / sms) * KB;
        const int parts = pick_ksplit(rows * j16, KB);
        // a split stage of more than one round is slow beyond this estimate (its many short tiles each end in
        // atomics): 1024 x 1024 x 16384 at 17 to 64 tokens took 56 to 82 us in the split form, 55 on the tiles
        if (rows * j16 * parts > sms) return false;
        split_cost += (KB + parts - 1) / parts;
    }
    return split_cost < tiles_cost;
}

// Four launches: x -> digits (clears the V-stage sums) | V-stage parts, the last part of each tile
// writes t = S*z and the per-token max |t| | t -> digits (clears the U-stage sums) | U-stage
// parts, the last part of each tile writes y.
template <typename IN_T, int NDX>
tsvd_status_t forward_small(const ForwardArgs& a, const SmallWs& w)
{
    tsvd_handle_s* h = a.h;
    const int KBv = h->V.C_pad / BLOCK_C, KBu = h->U.C_pad / BLOCK_C;
    const int Bp = (a.B + SMALL_TOK - 1) / SMALL_TOK * SMALL_TOK;
    const int j_tiles = Bp / SMALL_TOK;
    cudaStream_t st = a.stream;
    cudaError_t e;

    h->prof.begin(0, st);
    e = launch_digitise<IN_T, NDX, SMALL_TOK>((const IN_T*)a.x, a.ldx, a.B, h->N, KBv, nullptr, w.Dx, w.scale_x,
                                              w.zacc, w.zacc_ints, h->dev_status, h->prof.slot(0), st, a.gather);
    h->prof.end(st);
    if (e != cudaSuccess) return TSVD_E_CUDA;

    GemmParams p{};
    p.units = h->V.units; p.KB = KBv; p.R = h->K; p.D = w.Dx; p.B = a.B; p.status = h->dev_status;
    p.scale = w.scale_x; p.S = h->S; p.t = w.t; p.t_ld = h->V.R_pad;
    p.z_out = a.z_out; p.z_ld = h->K; p.z_int = (a.dtype == TSVD_I8);
    p.acc = w.zacc; p.acc_ld = h->V.R_pad;
    p.tmax = reinterpret_cast<unsigned*>(w.zacc + (size_t)Bp * NDX * h->V.R_pad);
    p.tile_done = w.zacc + (size_t)Bp * NDX * h->V.R_pad + Bp;
    p.tail = TAIL_T; p.stamp = h->prof.slot(1);
    const int v_tiles = h->V.R_pad / BLOCK_R;
    p.ksplit = pick_ksplit(v_tiles * j_tiles, KBv);
    h->prof.begin(1, st);
    e = launch_gemm<NDX, EPI_ACC, SMALL_TOK>(p, v_tiles, st);
    h->prof.end(st);
    if (e != cudaSuccess) return TSVD_E_CUDA;
    if (a.v_only) { *a.t_where = w.t; return TSVD_OK; }

    h->prof.begin(2, st);
    e = launch_digitise<float, ND_T, SMALL_TOK>(w.t, h->V.R_pad, a.B, h->K, KBu, p.tmax, w.Dt, w.scale_t, w.yacc,
                                                w.yacc_ints, h->dev_status, h->prof.slot(2), st);
    h->prof.end(st);
    if (e != cudaSuccess) return TSVD_E_CUDA;

    GemmParams q{};
    q.units = h->U.units; q.KB = KBu; q.R = h->M; q.D = w.Dt; q.B = a.B; q.status = h->dev_status;
    q.scale = w.scale_t; q.y = a.y; q.ldy = a.ldy; q.bias = h->bias;
    q.y_bf16 = (a.dtype == TSVD_BF16) && !a.out_f32;
    q.acc = w.yacc; q.acc_ld = h->U.R_pad;
    q.tile_done = w.yacc + (size_t)Bp * ND_T * h->U.R_pad;
    q.tail = TAIL_Y; q.stamp = h->prof.slot(3);
    const int u_tiles = h->U.R_pad / BLOCK_R;
    q.ksplit = pick_ksplit(u_tiles * j_tiles, KBu);
    h->prof.begin(3, st);
    e = launch_gemm<ND_T, EPI_ACC, SMALL_TOK>(q, u_tiles, st);
    h->prof.end(st);
    return e == cudaSuccess ? TSVD_OK : TSVD_E_CUDA;
}

}  // namespace

int tsvd_tensor_digits_x(tsvd_dtype_t dt, bool wide_x) { return digits_for_x(dt, wide_x); }
int tsvd_tensor_digits_t() { return ND_T; }

size_t tsvd_tensor_ws_bytes(const tsvd_handle_s* h, int B, tsvd_dtype_t dt, bool wide_x)
{
    if (B <= SMALL_MAX_B && prefer_split_form(h, B)) return carve_small(h, B, dt, wide_x, nullptr).total;
    return carve(h, B, dt, wide_x, nullptr).total;
}

// An upper bound of the scratch of any batch of up to B_max tokens (both forms grow with the batch; which of
// them a batch takes depends on the batch).
size_t tsvd_tensor_ws_bytes_upto(const tsvd_handle_s* h, int B_max, tsvd_dtype_t dt, bool wide_x)
{
    const size_t tiles = carve(h, B_max, dt, wide_x, nullptr).total;
    const size_t split = carve_small(h, B_max < SMALL_MAX_B ? B_max : SMALL_MAX_B, dt, wide_x, nullptr).total;
    return tiles > split ? tiles : split;
}

tsvd_status_t tsvd_forward_tensor(const ForwardArgs& a, void* ws)
{
    tsvd_handle_s* h = a.h;
    if (tsvd_mid_fits(h, a.B, a.dtype, a.wide_x)) return tsvd_forward_mid(a, ws);   // (its scratch is the smaller)
    if (a.B <= SMALL_MAX_B && prefer_split_form(h, a.B)) {
        // few tokens on few row tiles with long contractions: 16-token tiles, the contraction split across CTAs
        const SmallWs sw = carve_small(h, a.B, a.dtype, a.wide_x, ws);
        switch (a.dtype) {
            case TSVD_F32: return forward_small<float, 4>(a, sw);
            case TSVD_BF16: return a.wide_x ? forward_small<__nv_bfloat16, 4>(a, sw) : forward_small<__nv_bfloat16, 3>(a, sw);
            case TSVD_I8: return forward_small<int8_t, 1>(a, sw);
            default: return TSVD_E_DTYPE;
        }
    }
    const TensorWs w = carve(h, a.B, a.dtype, a.wide_x, ws);
    const bool wide_bf16 = a.dtype == TSVD_BF16 && a.wide_x;
    const bool narrow_i8 = a.dtype == TSVD_I8 && tokens_of_x_tile(h, 1, a.B) == TOK_I8_NARROW;
    const bool wide_x4 = (a.dtype == TSVD_F32 || wide_bf16) && tokens_of_x_tile(h, 4, a.B) == TOK_T_WIDE;
    const int KBv = h->V.C_pad / BLOCK_C, KBu = h->U.C_pad / BLOCK_C;
    cudaStream_t st = a.stream;
    cudaError_t e;

    // stage 0: activations -> digits
    unsigned long long* const stamp0 = h->prof.slot(0);
    h->prof.begin(0, st);
    switch (a.dtype) {
        case TSVD_F32:
            if (wide_x4)
                e = launch_digitise<float, 4, TOK_T_WIDE>((const float*)a.x, a.ldx, a.B, h->N, KBv, nullptr, w.Dx, w.scale_x,
                                                          nullptr, 0, h->dev_status, stamp0, st, a.gather);
            else
                e = launch_digitise<float, 4>((const float*)a.x, a.ldx, a.B, h->N, KBv, nullptr, w.Dx, w.scale_x, nullptr, 0,
                                              h->dev_status, stamp0, st, a.gather);
            break;
        case TSVD_BF16:
            if (wide_bf16 && wide_x4)
                e = launch_digitise<__nv_bfloat16, 4, TOK_T_WIDE>((const __nv_bfloat16*)a.x, a.ldx, a.B, h->N, KBv, nullptr,
                                                                  w.Dx, w.scale_x, nullptr, 0, h->dev_status, stamp0, st,
                                                                  a.gather);
            else if (wide_bf16)
                e = launch_digitise<__nv_bfloat16, 4>((const __nv_bfloat16*)a.x, a.ldx, a.B, h->N, KBv, nullptr, w.Dx,
                                                      w.scale_x, nullptr, 0, h->dev_status, stamp0, st, a.gather);
            else
                e = launch_digitise<__nv_bfloat16, 3>((const __nv_bfloat16*)a.x, a.ldx, a.B, h->N, KBv, nullptr, w.Dx,
                                                      w.scale_x, nullptr, 0, h->dev_status, stamp0, st, a.gather);
            break;
        case TSVD_I8:
            if (narrow_i8)
                e = launch_digitise<int8_t, 1, TOK_I8_NARROW>((const int8_t*)a.x, a.ldx, a.B, h->N, KBv, nullptr, w.Dx,
                                                              w.scale_x, nullptr, 0, h->dev_status, stamp0, st, a.gather);
            else
                e = launch_digitise<int8_t, 1>((const int8_t*)a.x, a.ldx, a.B, h->N, KBv, nullptr, w.Dx, w.scale_x,
                                               nullptr, 0, h->dev_status, stamp0, st, a.gather);
            break;
        default:
            return TSVD_E_DTYPE;
    }
    h->prof.end(st);
    if (e != cudaSuccess) return TSVD_E_CUDA;
    // stage 1: V-stage + S scale
    GemmParams p{};
    p.units = h->V.units; p.KB = KBv; p.R = h->K; p.D = w.Dx; p.scale = w.scale_x; p.B = a.B;
    p.S = h->S; p.t = w.t; p.t_ld = h->V.R_pad;
    p.z_out = a.z_out; p.z_ld = h->K; p.z_int = (a.dtype == TSVD_I8);
    p.status = h->dev_status; p.stamp = h->prof.slot(1);
    if (a.test_stall) { p.test_stall = 1; p.wait_limit = 16; }   // ~8 ms instead of ~2 s
    const int v_tiles = h->V.R_pad / BLOCK_R;
    h->prof.begin(1, st);
    if (wide_x4) e = launch_gemm<4, EPI_V, TOK_T_WIDE>(p, v_tiles, st);
    else if (a.dtype == TSVD_F32 || wide_bf16) e = launch_gemm<4, EPI_V>(p, v_tiles, st);
    else if (a.dtype == TSVD_BF16) e = launch_gemm<3, EPI_V>(p, v_tiles, st);
    else if (narrow_i8) e = launch_gemm<1, EPI_V, TOK_I8_NARROW>(p, v_tiles, st);
    else e = launch_gemm<1, EPI_V>(p, v_tiles, st);
    h->prof.end(st);
    if (e != cudaSuccess) return TSVD_E_CUDA;
    if (a.v_only) { *a.t_where = w.t; return TSVD_OK; }

    // stage 2: t -> digits (each token's scale comes from its own max |t|)
    h->prof.begin(2, st);
    const bool wide_t = tokens_of_t_tile(h, a.B) == TOK_T_WIDE;
    if (wide_t)
        e = launch_digitise<float, ND_T, TOK_T_WIDE>(w.t, h->V.R_pad, a.B, h->K, KBu, nullptr, w.Dt, w.scale_t, nullptr, 0,
                                                     h->dev_status, h->prof.slot(2), st);
    else
        e = launch_digitise<float, ND_T>(w.t, h->V.R_pad, a.B, h->K, KBu, nullptr, w.Dt, w.scale_t, nullptr, 0,
                                         h->dev_status, h->prof.slot(2), st);
    h->prof.end(st);
    if (e != cudaSuccess) return TSVD_E_CUDA;

    // stage 3: U-stage
    GemmParams q{};
    q.units = h->U.units; q.KB = KBu; q.R = h->M; q.D = w.Dt; q.scale = w.scale_t; q.B = a.B;
    q.y = a.y; q.ldy = a.ldy; q.status = h->dev_status; q.bias = h->bias; q.stamp = h->prof.slot(3);
    const int u_tiles = h->U.R_pad / BLOCK_R;
    const bool bf16_out = (a.dtype == TSVD_BF16) && !a.out_f32;
    h->prof.begin(3, st);
    if (wide_t) {
        if (bf16_out) e = launch_gemm<ND_T, EPI_U_BF16, TOK_T_WIDE>(q, u_tiles, st);
        else e = launch_gemm<ND_T, EPI_U_F32, TOK_T_WIDE>(q, u_tiles, st);
    } else if (bf16_out) {
        e = launch_gemm<ND_T, EPI_U_BF16>(q, u_tiles, st);
    } else {
        e = launch_gemm<ND_T, EPI_U_F32>(q, u_tiles, st);
    }
    h->prof.end(st);
    return e == cudaSuccess ? TSVD_OK : TSVD_E_CUDA;
}
