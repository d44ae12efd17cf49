// Decode path: y = U(diag(S)(V x)) for one to four tokens, bound by streaming the packed codes.
//
// For so few tokens a tensor-core tile is almost empty, and what matters is that every SM
// streams its share of the 2-bit codes (the whole of U and V is read once per forward) with as
// little fixed cost as possible.  Two launches, one per stage (Table S1 rows "V(.)" and "U(.)"):
// each CTA first turns the stage's input (x, or t = S*(V x)) into the same per-token fixed-point
// digits as the tensor-core path, in shared memory, then walks 32 rows of the packed matrix:
// a lane owns four rows of one 64-column group at a time, expands their codes to int8 with two
// byte permutes per eight entries and adds them to the digits with four-way integer dot
// products.  (Four rows per lane because every lane reads the same digits: a shared-memory load
// that all lanes aim at one address still takes its four passes, so each one has to feed as
// many dot products as the registers allow.)  All sums are exact integers, so the result does
// not depend on how the columns are split over the lanes and warps.
#include "digits.cuh"
#include "tsvd_internal.cuh"

namespace {

// threads per CTA: with one or two tokens the kernel waits on memory and wants many warps; with
// four the accumulators need the registers
__host__ __device__ constexpr int gemv_threads(int ntok) { return ntok <= 2 ? 512 : 256; }
constexpr int GEMV_RL = 8;          // lanes of a warp along the rows; the other four take different column groups
constexpr int GEMV_RPL = 4;         // rows per lane
constexpr int GEMV_CS = 32 / GEMV_RL;
constexpr int GEMV_ROWS = GEMV_RL * GEMV_RPL;   // rows per CTA
constexpr int GEMV_MAX_SMEM = 200 * 1024;

enum { STAGE_V = 0, STAGE_U = 1 };

struct GemvParams {
    const uint4* units;   // packed ternary operand
    int R, C, C_pad;      // logical rows and columns, padded columns
    const void* in;       // [B][ld_in]: activations (V-stage) or t (U-stage, fp32)
    int ld_in;
    int B;
    const float* S;       // V-stage: padded to R_pad
    void* out;            // V-stage: t fp32 [B][ld_out] (all padded rows); U-stage: y [B][ld_out]
    int ld_out;
    int out_bf16;
    void* z_out;          // V-stage, optional: [B][z_ld] int32 (z_int) or fp32
    int z_ld;
    int z_int;
};

// grid: R_pad / 32 CTAs of 256 threads.  Dynamic shared memory:
//   digits [NTOK][ND][C_pad] int8 | partial sums [warps][NTOK*ND][32 rows] int32 |
//   scale [NTOK] | per-warp maxima [warps][NTOK]
template <typename IN_T, int ND, int NTOK, int STAGE>
__global__ void __launch_bounds__(gemv_threads(NTOK))
ternary_gemv_kernel(const GemvParams p)
{
    extern __shared__ __align__(16) uint8_t smem[];
    constexpr int GEMV_THREADS = gemv_threads(NTOK), GEMV_WARPS = GEMV_THREADS / 32;
    constexpr bool kInt = sizeof(IN_T) == 1;
    static_assert(!kInt || ND == 1, "int8 activations are their own digit");
    int8_t* dig = reinterpret_cast<int8_t*>(smem);
    int* red = reinterpret_cast<int*>(smem + (size_t)NTOK * ND * p.C_pad);
    float* scale = reinterpret_cast<float*>(red + GEMV_WARPS * NTOK * ND * GEMV_ROWS);
    float* wmax = scale + NTOK;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const IN_T* in = reinterpret_cast<const IN_T*>(p.in);

    // lane = (column group within the pass, row); rows rsel, rsel + 8, .. of the CTA's 32; warp w
    // takes column groups 4w + csel, + 4 * warps, ..  The first codes are requested before anything
    // else, so that their trip from HBM overlaps with the digit conversion below.
    const int rsel = lane & (GEMV_RL - 1), csel = lane / GEMV_RL;
    const int row_base = blockIdx.x * GEMV_ROWS + rsel;
    const int n_groups = p.C_pad >> 6;
    auto load_units = [&](int g, uint4 (&uu)[GEMV_RPL]) {
#pragma unroll
        for (int j = 0; j < GEMV_RPL; ++j)
            uu[j] = g < n_groups ? __ldcs(p.units + tsvd_unit_index(row_base + j * GEMV_RL, g, p.C_pad))
                                 : make_uint4(0, 0, 0, 0);
    };
    int cg = GEMV_CS * warp + csel;
    uint4 u[GEMV_RPL];
    load_units(cg, u);
    // Both stages are launched as programmatic dependents of the kernel before them in the
    // stream: their CTAs may start, and request their first codes (which no kernel writes), while
    // that kernel still runs.  The stage's input (x, or t from the V-stage) is complete and
    // visible only after this wait, and the stage's output is written after it, so a kernel that
    // still reads t or y is never overtaken.  The next kernel in the stream may start likewise.
    pdl_wait();
    pdl_launch_dependents();

    // ---- the stage's input as fixed-point digits (every CTA makes its own copy).  A thread takes
    //      chunks of 16 consecutive columns; all loads of a pass are independent, so a pass costs
    //      about one trip to L2, and the first chunk of each token stays in registers between the
    //      maximum pass and the conversion pass ----
    const int n_chunks = p.C_pad >> 4;
    float keep[NTOK][16];
    float qscale[NTOK];
#pragma unroll
    for (int b = 0; b < NTOK; ++b) qscale[b] = 1.f;
    bool vec_ok[NTOK];
#pragma unroll
    for (int b = 0; b < NTOK; ++b)
        vec_ok[b] = ((reinterpret_cast<uintptr_t>(in + (size_t)b * p.ld_in)) & 15) == 0;
    if constexpr (!kInt) {
        float amax[NTOK];
#pragma unroll
        for (int b = 0; b < NTOK; ++b) amax[b] = 0.f;
        for (int ch = tid; ch < n_chunks; ch += GEMV_THREADS) {
#pragma unroll
            for (int b = 0; b < NTOK; ++b) {
                if (b < p.B) {
                    float v[16];
                    load16<IN_T>(in + (size_t)b * p.ld_in, ch * 16, p.C, vec_ok[b], v);
#pragma unroll
                    for (int e = 0; e < 16; ++e) amax[b] = fmaxf(amax[b], fabsf(v[e]));
                    if (ch == tid) {
#pragma unroll
                        for (int e = 0; e < 16; ++e) keep[b][e] = v[e];
                    }
                }
            }
        }
#pragma unroll
        for (int b = 0; b < NTOK; ++b) {
            for (int o = 16; o > 0; o >>= 1) amax[b] = fmaxf(amax[b], __shfl_xor_sync(0xffffffffu, amax[b], o));
            if (lane == 0) wmax[warp * NTOK + b] = amax[b];
        }
        __syncthreads();
#pragma unroll
        for (int b = 0; b < NTOK; ++b) {
            float m = 0.f;
#pragma unroll
            for (int w = 0; w < GEMV_WARPS; ++w) m = fmaxf(m, wmax[w * NTOK + b]);
            const int E = tsvd_quant_exponent(m);
            qscale[b] = tsvd_pow2(8 * ND - 2 - E);
            if (tid == 0) scale[b] = tsvd_pow2(E - (8 * ND - 2));   // value = q * scale
        }
    } else {
        if (tid < NTOK) scale[tid] = 1.f;
    }
    for (int ch = tid; ch < n_chunks; ch += GEMV_THREADS) {
#pragma unroll
        for (int b = 0; b < NTOK; ++b) {
            uint32_t dw[ND][4];
#pragma unroll
            for (int d = 0; d < ND; ++d)
#pragma unroll
                for (int g = 0; g < 4; ++g) dw[d][g] = 0u;
            if (b < p.B) {
                float v[16];
                if (!kInt && ch == tid) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) v[e] = keep[b][e];
                } else {
                    load16<IN_T>(in + (size_t)b * p.ld_in, ch * 16, p.C, vec_ok[b], v);
                }
                int q[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) q[e] = __float2int_rn(v[e] * qscale[b]);
                digits_of_16<ND>(q, dw);
            }
#pragma unroll
            for (int d = 0; d < ND; ++d)
                *reinterpret_cast<uint4*>(dig + (size_t)(b * ND + d) * p.C_pad + ch * 16) =
                    make_uint4(dw[d][0], dw[d][1], dw[d][2], dw[d][3]);
        }
    }
    __syncthreads();

    // ---- stream the codes ----
    int acc[GEMV_RPL][NTOK][ND];
#pragma unroll
    for (int j = 0; j < GEMV_RPL; ++j)
#pragma unroll
        for (int b = 0; b < NTOK; ++b)
#pragma unroll
            for (int d = 0; d < ND; ++d) acc[j][b][d] = 0;

    for (; cg < n_groups; cg += GEMV_CS * GEMV_WARPS) {
        uint4 un[GEMV_RPL];   // the next pass, in flight while this one is summed
        load_units(cg + GEMV_CS * GEMV_WARPS, un);
#pragma unroll
        for (int wi = 0; wi < 4; ++wi) {
            uint32_t e[GEMV_RPL][4];   // sixteen entries of each row as int8, in column order
#pragma unroll
            for (int j = 0; j < GEMV_RPL; ++j)
                tsvd_expand16(wi == 0 ? u[j].x : wi == 1 ? u[j].y : wi == 2 ? u[j].z : u[j].w, e[j]);
#pragma unroll
            for (int b = 0; b < NTOK; ++b) {
#pragma unroll
                for (int d = 0; d < ND; ++d) {
                    const uint4 xd = *reinterpret_cast<const uint4*>(dig + (size_t)(b * ND + d) * p.C_pad + cg * 64 + wi * 16);
#pragma unroll
                    for (int j = 0; j < GEMV_RPL; ++j) {
                        int s = acc[j][b][d];
                        s = __dp4a((int)e[j][0], (int)xd.x, s);
                        s = __dp4a((int)e[j][1], (int)xd.y, s);
                        s = __dp4a((int)e[j][2], (int)xd.z, s);
                        s = __dp4a((int)e[j][3], (int)xd.w, s);
                        acc[j][b][d] = s;
                    }
                }
            }
        }
#pragma unroll
        for (int j = 0; j < GEMV_RPL; ++j) u[j] = un[j];
    }

    // ---- add the lanes that took different column groups, then the warps ----
#pragma unroll
    for (int j = 0; j < GEMV_RPL; ++j)
#pragma unroll
        for (int b = 0; b < NTOK; ++b)
#pragma unroll
            for (int d = 0; d < ND; ++d) {
                int v = acc[j][b][d];
#pragma unroll
                for (int o = GEMV_RL; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if (csel == 0) red[(warp * NTOK * ND + b * ND + d) * GEMV_ROWS + j * GEMV_RL + rsel] = v;
            }
    __syncthreads();

    // ---- thread (token, row): digits -> fp32 -> the stage's output ----
    if (tid < NTOK * GEMV_ROWS) {
        const int b = tid / GEMV_ROWS, r = tid % GEMV_ROWS;
        const int orow = blockIdx.x * GEMV_ROWS + r;
        if (b < p.B) {
            int a[ND];
#pragma unroll
            for (int d = 0; d < ND; ++d) {
                int s = 0;
#pragma unroll
                for (int w = 0; w < GEMV_WARPS; ++w) s += red[(w * NTOK * ND + b * ND + d) * GEMV_ROWS + r];
                a[d] = s;
            }
            // lo and hi are exact 32-bit integers; their conversions and the fused multiply-add
            // round at 2^-24 of |hi|*65536 and |lo|
            float f;
            if constexpr (ND == 1) f = (float)a[0];
            else if constexpr (ND == 2) f = (float)(a[0] + (a[1] << 8));
            else {
                const int lo = a[0] + (a[1] << 8);
                int hi = a[2];
                if constexpr (ND == 4) hi += a[3] << 8;
                f = fmaf((float)hi, 65536.f, (float)lo);
            }
            const float val = f * scale[b];   // a power of two: exact
            if constexpr (STAGE == STAGE_V) {
                // the K multiplications (Table S1); padded rows have S = 0 and no codes
                reinterpret_cast<float*>(p.out)[(size_t)b * p.ld_out + orow] = p.S[orow] * val;
                if (p.z_out && orow < p.R) {
                    if (p.z_int) reinterpret_cast<int*>(p.z_out)[(size_t)b * p.z_ld + orow] = a[0];
                    else reinterpret_cast<float*>(p.z_out)[(size_t)b * p.z_ld + orow] = val;
                }
            } else if (orow < p.R) {
                if (p.out_bf16)
                    reinterpret_cast<__nv_bfloat16*>(p.out)[(size_t)b * p.ld_out + orow] = __float2bfloat16_rn(val);
                else
                    reinterpret_cast<float*>(p.out)[(size_t)b * p.ld_out + orow] = val;
            }
        }
    }
}

size_t gemv_smem_bytes(int nd, int ntok, int C_pad)
{
    const size_t warps = gemv_threads(ntok) / 32;
    return (size_t)ntok * nd * C_pad + warps * ntok * nd * GEMV_ROWS * sizeof(int) +
           (size_t)ntok * sizeof(float) + warps * ntok * sizeof(float);
}

template <typename IN_T, int ND, int NTOK, int STAGE>
cudaError_t launch_gemv(const GemvParams& p, int R_pad, cudaStream_t stream)
{
    static bool attr_set[64] = {};   // per instantiation and device
    const size_t smem = gemv_smem_bytes(ND, NTOK, p.C_pad);
    int dev = 0;
    cudaError_t e0 = cudaGetDevice(&dev);
    if (e0 != cudaSuccess) return e0;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(ternary_gemv_kernel<IN_T, ND, NTOK, STAGE>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, GEMV_MAX_SMEM);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    PdlLaunch cfg((unsigned)(R_pad / GEMV_ROWS), (unsigned)gemv_threads(NTOK), smem, stream);
    const cudaError_t e = cudaLaunchKernelEx(&cfg.cfg, ternary_gemv_kernel<IN_T, ND, NTOK, STAGE>, (const GemvParams)p);
    tsvd_count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename IN_T, int ND, int STAGE>
cudaError_t launch_gemv_tokens(const GemvParams& p, int R_pad, cudaStream_t stream)
{
    if (p.B == 1) return launch_gemv<IN_T, ND, 1, STAGE>(p, R_pad, stream);
    if (p.B == 2) return launch_gemv<IN_T, ND, 2, STAGE>(p, R_pad, stream);
    return launch_gemv<IN_T, ND, 4, STAGE>(p, R_pad, stream);
}

constexpr int ND_T = 4;   // digits of the intermediate t (fp32), as on the tensor-core path
inline int digits_for_x(tsvd_dtype_t dt) { return dt == TSVD_I8 ? 1 : dt == TSVD_BF16 ? 3 : 4; }

}  // namespace

bool tsvd_decode_fits(const tsvd_handle_s* h, int B, tsvd_dtype_t dt)
{
    if (B < 1 || B > TSVD_DECODE_MAX_B) return false;
    const int ntok = B == 3 ? 4 : B;
    return gemv_smem_bytes(digits_for_x(dt), ntok, h->V.C_pad) <= (size_t)GEMV_MAX_SMEM &&
           gemv_smem_bytes(ND_T, ntok, h->U.C_pad) <= (size_t)GEMV_MAX_SMEM;
}

size_t tsvd_decode_ws_bytes(const tsvd_handle_s* h, int B) { return (size_t)B * h->V.R_pad * sizeof(float); }

tsvd_status_t tsvd_forward_decode(const ForwardArgs& a, void* ws)
{
    tsvd_handle_s* h = a.h;
    cudaStream_t st = a.stream;
    float* t = reinterpret_cast<float*>(ws);

    GemvParams p{};
    p.units = h->V.units; p.R = h->K; p.C = h->N; p.C_pad = h->V.C_pad;
    p.in = a.x; p.ld_in = a.ldx; p.B = a.B; p.S = h->S;
    p.out = t; p.ld_out = h->V.R_pad;
    p.z_out = a.z_out; p.z_ld = h->K; p.z_int = (a.dtype == TSVD_I8);
    cudaError_t e;
    h->prof.begin(1, st);
    switch (a.dtype) {
        case TSVD_F32: e = launch_gemv_tokens<float, 4, STAGE_V>(p, h->V.R_pad, st); break;
        case TSVD_BF16: e = launch_gemv_tokens<__nv_bfloat16, 3, STAGE_V>(p, h->V.R_pad, st); break;
        case TSVD_I8: e = launch_gemv_tokens<int8_t, 1, STAGE_V>(p, h->V.R_pad, st); break;
        default: return TSVD_E_DTYPE;
    }
    h->prof.end(st);
    if (e != cudaSuccess) return TSVD_E_CUDA;

    GemvParams q{};
    q.units = h->U.units; q.R = h->M; q.C = h->K; q.C_pad = h->U.C_pad;
    q.in = t; q.ld_in = h->V.R_pad; q.B = a.B;
    q.out = a.y; q.ld_out = a.ldy;
    q.out_bf16 = (a.dtype == TSVD_BF16) && !a.out_f32;
    h->prof.begin(3, st);
    e = launch_gemv_tokens<float, ND_T, STAGE_U>(q, h->U.R_pad, st);
    h->prof.end(st);
    return e == cudaSuccess ? TSVD_OK : TSVD_E_CUDA;
}
