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
//   digitise(x)  ->  V-stage MMA  ->  epilogue: z = int * 2^e, t = S*z (the K multiplications),
//   per-token max|t|  ->  digitise(t)  ->  U-stage MMA  ->  epilogue: y = int * 2^e
#include "sm100_ptx.cuh"
#include "tsvd_internal.cuh"

namespace {

using namespace ptx;

constexpr int BLOCK_R = 128;   // ternary rows per CTA tile = MMA M
constexpr int BLOCK_C = 128;   // contraction elements per pipeline stage (one 128-byte swizzle row)
constexpr int UMMA_K = 32;     // contraction elements per kind::i8 instruction
constexpr int STAGES = 4;
constexpr int TMEM_COLS = 256;
constexpr int GEMM_THREADS = 192;  // warp 0: copies, warp 1: MMA issue, warps 2..5: expand + epilogue

// tokens per tile for nd digits: the MMA N extent is nd * tokens <= 256 and a multiple of 16
__host__ __device__ constexpr int tokens_per_tile(int nd) { return nd == 1 ? 256 : nd == 2 ? 128 : nd == 3 ? 80 : 64; }

constexpr int A_TILE_BYTES = BLOCK_R * BLOCK_C;          // expanded int8 operand, 16 KiB
constexpr int P_TILE_BYTES = BLOCK_R * BLOCK_C / 4;      // packed codes of that tile, 4 KiB
constexpr int B_TILE_BYTES_MAX = 256 * BLOCK_C;          // digit rows, up to 32 KiB
constexpr int STAGE_BYTES = A_TILE_BYTES + B_TILE_BYTES_MAX + P_TILE_BYTES;
constexpr int GEMM_SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;

// ---------------------------------------------------------------------------------------
// Digit matrix layout (scratch written by digitise_kernel, read by bulk copies):
// tiles of NT = nd*TOK rows x 128 contraction bytes, tile (jt, kb) at byte offset
// (jt*KB + kb) * NT*128.  Row (d*TOK + b_in) holds digit d of token jt*TOK + b_in.  Inside
// the tile, rows are 128 bytes with the 16-byte chunk index XORed with (row & 7): exactly the
// K-major 128-byte-swizzle operand layout, so a tile is one contiguous bulk copy.
// ---------------------------------------------------------------------------------------

template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <> __device__ __forceinline__ float to_float<int8_t>(int8_t v) { return (float)v; }

// One block per token slot b in [0, B_pad).  ND digits.  `amax_bits` (optional) holds the
// precomputed max |value| of each token as float bits; otherwise the block reduces it.
// For int8 input (ND == 1) the values are their own single digit and the scale is 1.
template <typename IN_T, int ND>
__global__ void __launch_bounds__(256)
digitise_kernel(const IN_T* __restrict__ in, int ld_in, int B, int C, int KB,
                const unsigned* __restrict__ amax_bits, int8_t* __restrict__ D, float* __restrict__ scale_out,
                unsigned* __restrict__ zero_me)
{
    constexpr int TOK = tokens_per_tile(ND);
    constexpr int NT = ND * TOK;
    constexpr bool kInt = sizeof(IN_T) == 1;
    const int b = blockIdx.x;
    const int jt = b / TOK, b_in = b % TOK;
    const bool live = b < B;
    const IN_T* row = in + (size_t)b * ld_in;
    __shared__ float red[8];
    __shared__ float s_qscale;

    if (zero_me && threadIdx.x == 0) zero_me[b] = 0u;

    if constexpr (!kInt) {
        float amax = 0.f;
        if (live) {
            if (amax_bits) {
                amax = __uint_as_float(amax_bits[b]);
            } else {
                for (int c = threadIdx.x; c < C; c += blockDim.x) amax = fmaxf(amax, fabsf(to_float<IN_T>(row[c])));
                for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
                if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
                __syncthreads();
                amax = red[0];
                for (int w = 1; w < (int)(blockDim.x >> 5); ++w) amax = fmaxf(amax, red[w]);
            }
        }
        if (threadIdx.x == 0) {
            // |v| <= amax < 2^E; quantise to q = rint(v * 2^(8ND-2-E)), so |q| <= 2^(8ND-2)
            int E = -90;
            if (amax > 0.f) {
                int e;
                (void)frexpf(amax, &e);
                E = max(e, -90);
            }
            s_qscale = exp2f((float)(8 * ND - 2 - E));
            scale_out[b] = exp2f((float)(E - (8 * ND - 2)));   // value = q * scale
        }
        __syncthreads();
    } else {
        if (threadIdx.x == 0) scale_out[b] = 1.f;
    }
    const float qscale = kInt ? 1.f : s_qscale;

    // each thread converts chunks of 16 consecutive contraction elements
    const int n_chunks = KB * 8;
    for (int ch = threadIdx.x; ch < n_chunks; ch += blockDim.x) {
        const int kb = ch >> 3, cc = ch & 7;
        const int c0 = ch * 16;
        uint32_t dig[ND][4];
#pragma unroll
        for (int d = 0; d < ND; ++d)
#pragma unroll
            for (int w = 0; w < 4; ++w) dig[d][w] = 0;
        if (live) {
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const int c = c0 + e;
                int q = 0;
                if (c < C) {
                    if constexpr (kInt) q = (int)row[c];
                    else q = __float2int_rn(to_float<IN_T>(row[c]) * qscale);
                }
#pragma unroll
                for (int d = 0; d < ND; ++d) {
                    int dv;
                    if (d == ND - 1) dv = q;                       // top digit: what is left
                    else { dv = (int)(int8_t)(q & 0xFF); q = (q - dv) >> 8; }
                    dig[d][e >> 2] |= (uint32_t)(dv & 0xFF) << (8 * (e & 3));
                }
            }
        }
        int8_t* tile = D + ((size_t)jt * KB + kb) * (size_t)(NT * 128);
#pragma unroll
        for (int d = 0; d < ND; ++d) {
            const int r = d * TOK + b_in;
            uint4 v = make_uint4(dig[d][0], dig[d][1], dig[d][2], dig[d][3]);
            *reinterpret_cast<uint4*>(tile + r * 128 + ((cc ^ (r & 7)) << 4)) = v;
        }
    }
}

// ---------------------------------------------------------------------------------------
// The contraction kernel.  CTA (rt, jt) computes the 128 x (ND*TOK) integer tile
//   acc[r, d*TOK + i] = sum_c T[rt*128 + r, c] * digit_d(token jt*TOK + i)[c]
// in tensor memory, then combines the digits and applies the stage's epilogue.
// ---------------------------------------------------------------------------------------
enum { EPI_V = 0, EPI_U_F32 = 1, EPI_U_BF16 = 2 };

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
    unsigned* tmax;       // EPI_V: per-token max |t| as float bits (atomicMax)
    void* z_out;          // EPI_V: optional [B][z_ld]: int32 when z_int, else fp32
    int z_ld;
    int z_int;
    void* y;              // EPI_U_*: out [B][ldy]
    int ldy;
    int* status;          // device error word
};

template <int ND, int EPI>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
ternary_mma_kernel(const GemmParams p)
{
    constexpr int TOK = tokens_per_tile(ND);
    constexpr int NT = ND * TOK;
    constexpr uint32_t B_TILE_BYTES = NT * BLOCK_C;
    constexpr uint32_t IDESC = umma_idesc_s8(BLOCK_R, NT);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* a_tiles = smem;                                   // STAGES x 16 KiB, 1024-aligned
    uint8_t* b_tiles = smem + STAGES * A_TILE_BYTES;           // STAGES x 32 KiB, 1024-aligned
    uint8_t* p_tiles = b_tiles + STAGES * B_TILE_BYTES_MAX;    // STAGES x 4 KiB
    uint64_t* bars = reinterpret_cast<uint64_t*>(p_tiles + STAGES * P_TILE_BYTES);
    uint64_t* full_bar = bars;                 // copies landed (packed codes + digit tile)
    uint64_t* aready_bar = bars + STAGES;      // expanded operand written
    uint64_t* empty_bar = bars + 2 * STAGES;   // MMAs that read the stage have completed
    uint64_t* acc_bar = bars + 3 * STAGES;     // all MMAs of the tile have completed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 3 * STAGES + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rt = blockIdx.x, jt = blockIdx.y;
    const int KB = p.KB;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&aready_bar[s], 4);   // one arrival per expander warp
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(acc_bar, 1);
        *abort_flag = 0;
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

    if (warp == 0) {
        // ---- copy producer: packed codes of the A tile and the digit tile, per stage ----
        if (lane == 0) {
            const uint8_t* p_src = reinterpret_cast<const uint8_t*>(p.units) + (size_t)rt * KB * P_TILE_BYTES;
            const int8_t* d_src = p.D + (size_t)jt * KB * B_TILE_BYTES;
            int issued = 0;
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % STAGES;
                const uint32_t use = kb / STAGES;
                if (use > 0 && !mbar_wait(&empty_bar[s], (use - 1) & 1, abort_flag)) break;
                issued = kb + 1;
                mbar_arrive_expect_tx(&full_bar[s], P_TILE_BYTES + B_TILE_BYTES);
                bulk_g2s(p_tiles + s * P_TILE_BYTES, p_src + (size_t)kb * P_TILE_BYTES, P_TILE_BYTES, &full_bar[s]);
                bulk_g2s(b_tiles + s * B_TILE_BYTES_MAX, d_src + (size_t)kb * B_TILE_BYTES, B_TILE_BYTES,
                         &full_bar[s]);
            }
            if (*abort_flag) {
                // a wait gave up somewhere: let this CTA's own copies land before it exits (bounded)
                for (int kb = max(0, issued - STAGES); kb < issued; ++kb) {
                    uint64_t* bar = &full_bar[kb % STAGES];
                    const uint32_t ph = (kb / STAGES) & 1;
                    for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(bar, ph); ++spin) {}
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issue: one thread ----
        if (lane == 0) {
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % STAGES;
                const uint32_t ph = (kb / STAGES) & 1;
                if (!mbar_wait(&full_bar[s], ph, abort_flag)) break;
                if (!mbar_wait(&aready_bar[s], ph, abort_flag)) break;
                tc_fence_after_sync();
                const uint64_t a_desc = umma_desc_k_sw128(smem_u32(a_tiles + s * A_TILE_BYTES));
                const uint64_t b_desc = umma_desc_k_sw128(smem_u32(b_tiles + s * B_TILE_BYTES_MAX));
#pragma unroll
                for (int k = 0; k < BLOCK_C / UMMA_K; ++k) {
                    // advance both operands by 32 bytes inside the swizzled 128-byte rows
                    umma_s8_ss(tmem_base, a_desc + (uint64_t)(k * (UMMA_K >> 4)),
                               b_desc + (uint64_t)(k * (UMMA_K >> 4)), IDESC, (kb | k) != 0);
                }
                umma_commit(&empty_bar[s]);   // frees the stage when these MMAs are done
            }
            umma_commit(acc_bar);
        }
    } else {
        // ---- expanders: thread = row of the tile ----
        const int r = threadIdx.x - 64;   // 0..127
        for (int kb = 0; kb < KB; ++kb) {
            const int s = kb % STAGES;
            const uint32_t ph = (kb / STAGES) & 1;
            if (!mbar_wait(&full_bar[s], ph, abort_flag)) break;
            const uint4* packed = reinterpret_cast<const uint4*>(p_tiles + s * P_TILE_BYTES);
            uint8_t* a_row = a_tiles + s * A_TILE_BYTES + r * 128;
#pragma unroll
            for (int g = 0; g < 2; ++g) {
                const uint4 u = packed[g * 128 + r];
                const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
                for (int wi = 0; wi < 4; ++wi) {
                    uint32_t o[4];
                    tsvd_expand16(w[wi], o);
                    const int chunk = g * 4 + wi;
                    *reinterpret_cast<uint4*>(a_row + ((chunk ^ (r & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
            fence_proxy_async_smem();   // generic-proxy stores -> visible to the MMA's async reads
            __syncwarp();
            if (lane == 0) mbar_arrive(&aready_bar[s]);
        }

        // ---- epilogue: this warp owns tensor-memory lanes 32*(warp%4) .. +31 ----
        const int lane_grp = warp & 3;
        const int row_in = lane_grp * 32 + lane;
        const int row = rt * BLOCK_R + row_in;
        const bool ok = mbar_wait(acc_bar, 0, abort_flag);
        tc_fence_after_sync();
        if (ok) {
            const uint32_t t_lane = tmem_base + ((uint32_t)(lane_grp * 32) << 16);
            float s_row = 0.f;
            if constexpr (EPI == EPI_V) s_row = p.S[row];
            for (int g = 0; g < TOK / 16; ++g) {
                uint32_t acc[ND][16];
#pragma unroll
                for (int d = 0; d < ND; ++d) tmem_ld16(t_lane + (uint32_t)(d * TOK + g * 16), acc[d]);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int b = jt * TOK + g * 16 + i;
                    long long v = (long long)(int)acc[0][i];
#pragma unroll
                    for (int d = 1; d < ND; ++d) v += (long long)(int)acc[d][i] << (8 * d);
                    const bool live = b < p.B;   // uniform across the warp
                    const float sc = live ? p.scale[b] : 0.f;
                    const float val = __ll2float_rn(v) * sc;   // sc is a power of two: one rounding
                    if constexpr (EPI == EPI_V) {
                        const float tv = s_row * val;           // the K multiplications (Table S1)
                        if (live) {
                            p.t[(size_t)b * p.t_ld + row] = tv;
                            if (p.z_out && row < p.R) {
                                if (p.z_int) reinterpret_cast<int*>(p.z_out)[(size_t)b * p.z_ld + row] = (int)v;
                                else reinterpret_cast<float*>(p.z_out)[(size_t)b * p.z_ld + row] = val;
                            }
                            const unsigned m = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(tv)));
                            if (lane == 0) atomicMax(&p.tmax[b], m);
                        }
                    } else if constexpr (EPI == EPI_U_F32) {
                        if (live && row < p.R) reinterpret_cast<float*>(p.y)[(size_t)b * p.ldy + row] = val;
                    } else {
                        if (live && row < p.R)
                            reinterpret_cast<__nv_bfloat16*>(p.y)[(size_t)b * p.ldy + row] = __float2bfloat16_rn(val);
                    }
                }
            }
        }
    }

    // ---- teardown ----
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) atomicExch(p.status, 1);
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

template <typename IN_T, int ND>
cudaError_t launch_digitise(const IN_T* in, int ld_in, int B, int C, int KB, const unsigned* amax_bits,
                            int8_t* D, float* scale, unsigned* zero_me, int* B_pad_out, cudaStream_t stream)
{
    constexpr int TOK = tokens_per_tile(ND);
    const int B_pad = (B + TOK - 1) / TOK * TOK;
    digitise_kernel<IN_T, ND><<<B_pad, 256, 0, stream>>>(in, ld_in, B, C, KB, amax_bits, D, scale, zero_me);
    tsvd_count_launch();
    if (B_pad_out) *B_pad_out = B_pad;
    return cudaGetLastError();
}

template <int ND, int EPI>
cudaError_t launch_gemm(const GemmParams& p, int row_tiles, cudaStream_t stream)
{
    constexpr int TOK = tokens_per_tile(ND);
    static bool attr_set[64] = {};   // per instantiation and device
    int dev = 0;
    cudaError_t e0 = cudaGetDevice(&dev);
    if (e0 != cudaSuccess) return e0;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(ternary_mma_kernel<ND, EPI>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_BYTES);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    dim3 grid(row_tiles, (p.B + TOK - 1) / TOK);
    ternary_mma_kernel<ND, EPI><<<grid, GEMM_THREADS, GEMM_SMEM_BYTES, stream>>>(p);
    tsvd_count_launch();
    return cudaGetLastError();
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// digit counts: int8 activations are their own single digit; bf16 needs 3 (22-bit fixed
// point holds every bf16 value within 2^-12 of the token's largest exactly); fp32 and the
// intermediate t use 4 (30 bits).
inline int digits_for_x(tsvd_dtype_t dt) { return dt == TSVD_I8 ? 1 : dt == TSVD_BF16 ? 3 : 4; }
constexpr int ND_T = 4;

struct TensorWs {
    int8_t* Dx; float* scale_x; float* t; unsigned* tmax; int8_t* Dt; float* scale_t;
    size_t total;
};

TensorWs carve(const tsvd_handle_s* h, int B, tsvd_dtype_t dt, void* base)
{
    const int ndx = digits_for_x(dt);
    const int tokx = tokens_per_tile(ndx), tokt = tokens_per_tile(ND_T);
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

size_t tsvd_tensor_ws_bytes(const tsvd_handle_s* h, int B, tsvd_dtype_t dt)
{
    return carve(h, B, dt, nullptr).total;
}

tsvd_status_t tsvd_forward_tensor(const ForwardArgs& a, void* ws)
{
    tsvd_handle_s* h = a.h;
    const TensorWs w = carve(h, a.B, a.dtype, ws);
    const int KBv = h->V.C_pad / BLOCK_C, KBu = h->U.C_pad / BLOCK_C;
    cudaStream_t st = a.stream;
    cudaError_t e;

    // stage 0: activations -> digits (also clears the per-token max of t)
    h->prof.begin(0, st);
    switch (a.dtype) {
        case TSVD_F32:
            e = launch_digitise<float, 4>((const float*)a.x, a.ldx, a.B, h->N, KBv, nullptr, w.Dx, w.scale_x, w.tmax,
                                          nullptr, st);
            break;
        case TSVD_BF16:
            e = launch_digitise<__nv_bfloat16, 3>((const __nv_bfloat16*)a.x, a.ldx, a.B, h->N, KBv, nullptr, w.Dx,
                                                  w.scale_x, w.tmax, nullptr, st);
            break;
        case TSVD_I8:
            e = launch_digitise<int8_t, 1>((const int8_t*)a.x, a.ldx, a.B, h->N, KBv, nullptr, w.Dx, w.scale_x,
                                           w.tmax, nullptr, st);
            break;
        default:
            return TSVD_E_DTYPE;
    }
    h->prof.end(st);
    if (e != cudaSuccess) return TSVD_E_CUDA;
    // stage 1: V-stage + S scale
    GemmParams p{};
    p.units = h->V.units; p.KB = KBv; p.R = h->K; p.D = w.Dx; p.scale = w.scale_x; p.B = a.B;
    p.S = h->S; p.t = w.t; p.t_ld = h->V.R_pad; p.tmax = w.tmax;
    p.z_out = a.z_out; p.z_ld = h->K; p.z_int = (a.dtype == TSVD_I8);
    p.status = h->dev_status;
    const int v_tiles = h->V.R_pad / BLOCK_R;
    h->prof.begin(1, st);
    if (a.dtype == TSVD_F32) e = launch_gemm<4, EPI_V>(p, v_tiles, st);
    else if (a.dtype == TSVD_BF16) e = launch_gemm<3, EPI_V>(p, v_tiles, st);
    else e = launch_gemm<1, EPI_V>(p, v_tiles, st);
    h->prof.end(st);
    if (e != cudaSuccess) return TSVD_E_CUDA;

    // stage 2: t -> digits, using the per-token max gathered by the V-stage epilogue
    h->prof.begin(2, st);
    e = launch_digitise<float, ND_T>(w.t, h->V.R_pad, a.B, h->K, KBu, w.tmax, w.Dt, w.scale_t, nullptr, nullptr, st);
    h->prof.end(st);
    if (e != cudaSuccess) return TSVD_E_CUDA;

    // stage 3: U-stage
    GemmParams q{};
    q.units = h->U.units; q.KB = KBu; q.R = h->M; q.D = w.Dt; q.scale = w.scale_t; q.B = a.B;
    q.y = a.y; q.ldy = a.ldy; q.status = h->dev_status;
    const int u_tiles = h->U.R_pad / BLOCK_R;
    const bool bf16_out = (a.dtype == TSVD_BF16) && !a.out_f32;
    h->prof.begin(3, st);
    if (bf16_out) e = launch_gemm<ND_T, EPI_U_BF16>(q, u_tiles, st);
    else e = launch_gemm<ND_T, EPI_U_F32>(q, u_tiles, st);
    h->prof.end(st);
    return e == cudaSuccess ? TSVD_OK : TSVD_E_CUDA;
}
