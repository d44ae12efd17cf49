// Support for the convolution forms of a TSVD layer (Section "TSVD in Convolution Layer"): after
// the kernel has been reshaped to one of the four matrices of Eq. 5 and decomposed, V(.) and U(.)
// are themselves convolutions (with kernels [K1,K2] and [1,1], or [1,1] and [K1,K2], or [1,K2] and
// [K1,1], or [K1,1] and [1,K2]) and diag(s)(.) is a channel-wise scale.  A convolution with a ternary
// kernel is the ternary matrix product of this library applied to the patches of its input, so the
// two pieces needed are a patch gather and an entry point that runs one ternary stage with its scale.
#include "tsvd_internal.cuh"

namespace {

// out[(n, ho, wo)][(a, b, c)] = x[n, ho*sh + a*dh - ph, wo*sw + b*dw - pw, c]  (zero outside the image)
// For one output pixel and one kernel position the C channels are contiguous in the image and in the
// patch, so the gather is a set of straight copies.  A block takes whole output pixels (its index
// arithmetic once per pixel); its threads take the pixel's chunks of VEC channels: 16 bytes each when
// the channel run, the two base pointers and the patch stride allow it, else one element.
template <typename T, int VEC>
__global__ void im2col_nhwc_kernel(const T* __restrict__ x, int H, int W, int C, int k1, int k2, int sh, int sw, int ph,
                                   int pw, int dh, int dw, int Ho, int Wo, T* __restrict__ out, long long ld_out,
                                   long long rows)
{
    struct alignas(sizeof(T) * VEC) Chunk { T v[VEC]; };
    const int cpi = C / VEC;               // chunks per (pixel, kernel position)
    const int per_row = k1 * k2 * cpi;     // chunks per output pixel
    for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
        const int wo = (int)(row % Wo);
        const long long r2 = row / Wo;
        const int ho = (int)(r2 % Ho);
        const long long n = r2 / Ho;
        T* dst = out + row * ld_out;
        for (int j = threadIdx.x; j < per_row; j += blockDim.x) {
            const int ab = j / cpi, ch = j - ab * cpi;
            const int a = ab / k2, b = ab - a * k2;
            const int h = ho * sh + a * dh - ph, w = wo * sw + b * dw - pw;
            Chunk c;
#pragma unroll
            for (int e = 0; e < VEC; ++e) c.v[e] = static_cast<T>(0.0f);
            if (h >= 0 && h < H && w >= 0 && w < W)
                c = *reinterpret_cast<const Chunk*>(x + ((n * H + h) * W + w) * C + (long long)ch * VEC);
            *reinterpret_cast<Chunk*>(dst + (long long)ab * C + (long long)ch * VEC) = c;
        }
    }
}

template <typename T>
cudaError_t launch_im2col(const void* x, int H, int W, int C, int k1, int k2, int sh, int sw, int ph, int pw, int dh, int dw,
                          int Ho, int Wo, void* out, long long ld_out, long long rows, cudaStream_t st)
{
    constexpr int VEC = 16 / (int)sizeof(T);
    const bool wide = C % VEC == 0 && ld_out % VEC == 0 && (((uintptr_t)x | (uintptr_t)out) & 15) == 0;
    const long long per_row = (long long)k1 * k2 * (wide ? C / VEC : C);
    const unsigned threads = (unsigned)(per_row >= 256 ? 256 : (per_row + 31) / 32 * 32);
    const unsigned blocks = (unsigned)(rows < 148LL * 64 ? rows : 148LL * 64);
    if (wide)
        im2col_nhwc_kernel<T, VEC><<<blocks, threads, 0, st>>>((const T*)x, H, W, C, k1, k2, sh, sw, ph, pw, dh, dw, Ho, Wo,
                                                               (T*)out, ld_out, rows);
    else
        im2col_nhwc_kernel<T, 1><<<blocks, threads, 0, st>>>((const T*)x, H, W, C, k1, k2, sh, sw, ph, pw, dh, dw, Ho, Wo,
                                                             (T*)out, ld_out, rows);
    return cudaGetLastError();
}

}  // namespace

extern "C" tsvd_status_t tsvd_im2col(const void* x, tsvd_dtype_t dtype, int n_img, int H, int W, int C, int k1, int k2,
                                     int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w, void* out,
                                     long long ld_out, void* stream)
{
    if (!x || !out) return TSVD_E_NULL;
    if (n_img < 1 || H < 1 || W < 1 || C < 1 || k1 < 1 || k2 < 1 || stride_h < 1 || stride_w < 1 || pad_h < 0 || pad_w < 0 ||
        dil_h < 1 || dil_w < 1)
        return TSVD_E_SHAPE;
    const int Ho = (H + 2 * pad_h - dil_h * (k1 - 1) - 1) / stride_h + 1;
    const int Wo = (W + 2 * pad_w - dil_w * (k2 - 1) - 1) / stride_w + 1;
    if (Ho < 1 || Wo < 1 || ld_out < (long long)k1 * k2 * C) return TSVD_E_SHAPE;
    const long long rows = (long long)n_img * Ho * Wo;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e;
    switch (dtype) {
        case TSVD_F32:
            e = launch_im2col<float>(x, H, W, C, k1, k2, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w, Ho, Wo, out, ld_out, rows, st);
            break;
        case TSVD_BF16:
            e = launch_im2col<__nv_bfloat16>(x, H, W, C, k1, k2, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w, Ho, Wo, out, ld_out,
                                             rows, st);
            break;
        case TSVD_I8:
            e = launch_im2col<int8_t>(x, H, W, C, k1, k2, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w, Ho, Wo, out, ld_out, rows, st);
            break;
        default:
            return TSVD_E_DTYPE;
    }
    tsvd_count_launch();
    return e == cudaSuccess ? TSVD_OK : TSVD_E_CUDA;
}
