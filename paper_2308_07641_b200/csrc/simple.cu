// CUDA-core kernels for the TSVD map: correctness-first, any shape, any batch.
//
// One generic kernel computes  out[b, r] = sum_c T[r, c] * in[b, c]  for a packed ternary
// matrix T, by additions and subtractions at the nonzero codes only (Table S1 rows "V(.)"
// and "U(.)").  It is launched twice per forward: on V with the activations (the epilogue
// then applies the K multiplications of the "diag(s)(.)" row), and on U with S*(V x).
#include "tsvd_internal.cuh"

namespace {

constexpr int TB = 8;  // tokens per block

template <typename T> struct Acc { using type = double; };
template <> struct Acc<int8_t> { using type = int; };

template <typename T> __device__ __forceinline__ float load_as_float(const T* p);
template <> __device__ __forceinline__ float load_as_float<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float load_as_float<__nv_bfloat16>(const __nv_bfloat16* p)
{
    return __bfloat162float(*p);
}

enum Epilogue { EPI_SCALE_TO_T = 0, EPI_Y_F32 = 1, EPI_Y_BF16 = 2 };

// grid: (R_pad/128, ceil(B/TB)); block: 128 threads, thread r owns row rt*128 + r.
template <typename IN_T, int EPI>
__global__ void __launch_bounds__(128)
ternary_rows_kernel(const uint4* __restrict__ units, int R, int C, int C_pad,
                    const IN_T* __restrict__ in, int ld_in, int B,
                    const float* __restrict__ S, void* __restrict__ out, int ld_out,
                    void* __restrict__ z_out, int z_ld,   // S: the scales (V-stage) or the optional bias (U-stage)
                    unsigned long long* __restrict__ stamp)
{
    tsvd_stamp_begin(stamp);
    constexpr bool kInt = sizeof(IN_T) == 1;
    using acc_t = typename Acc<IN_T>::type;
    using part_t = typename std::conditional<kInt, int, float>::type;
    __shared__ part_t xs[TB][TSVD_COL_GROUP];

    const int r_in = threadIdx.x;
    const int row = blockIdx.x * TSVD_ROW_TILE + r_in;
    const int b0 = blockIdx.y * TB;
    const int n_groups = C_pad / TSVD_COL_GROUP;
    const uint4* my_units = units + (size_t)blockIdx.x * (size_t)n_groups * 128 + r_in;

    acc_t acc[TB];
#pragma unroll
    for (int t = 0; t < TB; ++t) acc[t] = 0;

    for (int cg = 0; cg < n_groups; ++cg) {
        __syncthreads();
        for (int i = threadIdx.x; i < TB * TSVD_COL_GROUP; i += blockDim.x) {
            const int t = i / TSVD_COL_GROUP, c = i % TSVD_COL_GROUP;
            const int col = cg * TSVD_COL_GROUP + c;
            part_t v = 0;
            if (b0 + t < B && col < C) {
                if constexpr (kInt) v = (int)in[(size_t)(b0 + t) * ld_in + col];
                else v = load_as_float<IN_T>(in + (size_t)(b0 + t) * ld_in + col);
            }
            xs[t][c] = v;
        }
        __syncthreads();
        const uint4 u = my_units[(size_t)cg * 128];
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
        part_t part[TB];
#pragma unroll
        for (int t = 0; t < TB; ++t) part[t] = 0;
#pragma unroll
        for (int wi = 0; wi < 4; ++wi) {
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                // one addition or subtraction per nonzero code, nothing for a zero (no multiply)
                const uint32_t code = (w[wi] >> tsvd_entry_shift(e)) & 3u;
                const int c = wi * 16 + e;
#pragma unroll
                for (int t = 0; t < TB; ++t) {
                    const part_t xv = xs[t][c];
                    part[t] += (code & 1u) ? ((code & 2u) ? -xv : xv) : (part_t)0;
                }
            }
        }
#pragma unroll
        for (int t = 0; t < TB; ++t) acc[t] += (acc_t)part[t];
    }

    if (row >= R) { tsvd_stamp_end(stamp); return; }
#pragma unroll
    for (int t = 0; t < TB; ++t) {
        const int b = b0 + t;
        if (b >= B) break;
        if constexpr (EPI == EPI_SCALE_TO_T) {
            float z;
            if constexpr (kInt) {
                if (z_out) reinterpret_cast<int*>(z_out)[(size_t)b * z_ld + row] = acc[t];
                z = (float)acc[t];
            } else {
                z = (float)acc[t];
                if (z_out) reinterpret_cast<float*>(z_out)[(size_t)b * z_ld + row] = z;
            }
            reinterpret_cast<float*>(out)[(size_t)b * ld_out + row] = S[row] * z;
        } else {
            // the optional bias is added in fp32 before the one rounding to the output type
            const float yv = S ? (float)acc[t] + S[row] : (float)acc[t];
            if constexpr (EPI == EPI_Y_F32)
                reinterpret_cast<float*>(out)[(size_t)b * ld_out + row] = yv;
            else
                reinterpret_cast<__nv_bfloat16*>(out)[(size_t)b * ld_out + row] = __float2bfloat16_rn(yv);
        }
    }
    tsvd_stamp_end(stamp);
}

template <typename IN_T, int EPI>
cudaError_t launch(const PackedMat& pm, const IN_T* in, int ld_in, int B, const float* S, void* out,
                   int ld_out, void* z_out, int z_ld, cudaStream_t stream, unsigned long long* stamp = nullptr)
{
    dim3 grid(pm.R_pad / TSVD_ROW_TILE, (B + TB - 1) / TB);
    ternary_rows_kernel<IN_T, EPI><<<grid, 128, 0, stream>>>(pm.units, pm.R, pm.C, pm.C_pad, in, ld_in,
                                                             B, S, out, ld_out, z_out, z_ld, stamp);
    tsvd_count_launch();
    return cudaGetLastError();
}

}  // namespace

size_t tsvd_simple_ws_bytes(const tsvd_handle_s* h, int B)
{
    return (size_t)B * (size_t)h->V.R_pad * sizeof(float);
}

tsvd_status_t tsvd_forward_simple(const ForwardArgs& a)
{
    tsvd_handle_s* h = a.h;
    cudaError_t e;
    unsigned long long* const stamp_v = h->prof.slot(1);
    h->prof.begin(1, a.stream);
    // V-stage + S-stage: t[b,k] = S[k] * sum_n V[k,n] x[b,n]
    switch (a.dtype) {
        case TSVD_F32:
            e = launch<float, EPI_SCALE_TO_T>(h->V, (const float*)a.x, a.ldx, a.B, h->S, a.t, a.t_ld,
                                              a.z_out, h->K, a.stream, stamp_v);
            break;
        case TSVD_BF16:
            e = launch<__nv_bfloat16, EPI_SCALE_TO_T>(h->V, (const __nv_bfloat16*)a.x, a.ldx, a.B, h->S,
                                                      a.t, a.t_ld, a.z_out, h->K, a.stream, stamp_v);
            break;
        case TSVD_I8:
            e = launch<int8_t, EPI_SCALE_TO_T>(h->V, (const int8_t*)a.x, a.ldx, a.B, h->S, a.t, a.t_ld,
                                               a.z_out, h->K, a.stream, stamp_v);
            break;
        default:
            return TSVD_E_DTYPE;
    }
    h->prof.end(a.stream);
    if (e != cudaSuccess) return TSVD_E_CUDA;
    if (a.v_only) { *a.t_where = a.t; return TSVD_OK; }
    h->prof.begin(3, a.stream);
    // U-stage: y[b,m] = sum_k U[m,k] t[b,k]
    const bool bf16_out = (a.dtype == TSVD_BF16) && !a.out_f32;
    unsigned long long* const stamp_u = h->prof.slot(3);
    if (bf16_out)
        e = launch<float, EPI_Y_BF16>(h->U, a.t, a.t_ld, a.B, h->bias, a.y, a.ldy, nullptr, 0, a.stream, stamp_u);
    else
        e = launch<float, EPI_Y_F32>(h->U, a.t, a.t_ld, a.B, h->bias, a.y, a.ldy, nullptr, 0, a.stream, stamp_u);
    h->prof.end(a.stream);
    return e == cudaSuccess ? TSVD_OK : TSVD_E_CUDA;
}

// ---------------------------------------------------------------------------------------
// tsvd_forward_static: the same two kernels with the intermediate S*(V x) in a fixed
// array that is part of the library image, for callers that must not allocate.
// ---------------------------------------------------------------------------------------
#include <mutex>

// One array per device that loads the library.  In host code this name is only a handle
// for the runtime's symbol table, never a device address: the address each device uses
// is fetched with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[TSVD_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
float* g_static_ptr[kMaxDevices] = {};

// Device address of g_static_scratch on the CURRENT device (looked up once per device).
tsvd_status_t static_scratch_for(int device, float** out)
{
    if (device < 0 || device >= kMaxDevices) return TSVD_E_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) { (void)cudaGetLastError(); return TSVD_E_CUDA; }
        g_static_ptr[device] = reinterpret_cast<float*>(p);
    }
    *out = g_static_ptr[device];
    return TSVD_OK;
}
}  // namespace

extern "C" tsvd_status_t tsvd_forward_static(tsvd_handle_t h, const void* x, void* y, int B,
                                             tsvd_dtype_t dtype, void* stream)
{
    if (!h || !x || !y) return TSVD_E_NULL;
    if (B < 1) return TSVD_E_SHAPE;
    if (dtype != TSVD_F32 && dtype != TSVD_BF16 && dtype != TSVD_I8) return TSVD_E_DTYPE;
    if (((uintptr_t)x & 15) || ((uintptr_t)y & 15)) return TSVD_E_ALIGN;
    const size_t need = (size_t)B * (size_t)h->V.R_pad * sizeof(float);
    if (need > (size_t)TSVD_STATIC_SCRATCH_BYTES) return TSVD_E_TOOBIG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return TSVD_E_CUDA; }
    if (dev != h->device) return TSVD_E_CUDA;
    float* t = nullptr;
    tsvd_status_t st = static_scratch_for(dev, &t);
    if (st != TSVD_OK) return st;

    cudaStream_t s = (cudaStream_t)stream;
    const int t_ld = h->V.R_pad;
    cudaError_t e;
    if (dtype == TSVD_F32)
        e = launch<float, EPI_SCALE_TO_T>(h->V, (const float*)x, h->N, B, h->S, t, t_ld, nullptr, 0, s);
    else if (dtype == TSVD_BF16)
        e = launch<__nv_bfloat16, EPI_SCALE_TO_T>(h->V, (const __nv_bfloat16*)x, h->N, B, h->S, t, t_ld,
                                                  nullptr, 0, s);
    else
        e = launch<int8_t, EPI_SCALE_TO_T>(h->V, (const int8_t*)x, h->N, B, h->S, t, t_ld, nullptr, 0, s);
    if (e != cudaSuccess) return TSVD_E_CUDA;
    if (dtype == TSVD_BF16)
        e = launch<float, EPI_Y_BF16>(h->U, t, t_ld, B, h->bias, y, h->M, nullptr, 0, s);
    else
        e = launch<float, EPI_Y_F32>(h->U, t, t_ld, B, h->bias, y, h->M, nullptr, 0, s);
    return e == cudaSuccess ? TSVD_OK : TSVD_E_CUDA;
}
