// Support for the convolution forms of a TSVD layer (Section "TSVD in Convolution Layer"): after
// the kernel has been reshaped to one of the four matrices of Eq. 5 and decomposed, V(.) and U(.)
// are themselves convolutions (with kernels [K1,K2] and [1,1], or [1,1] and [K1,K2], or [1,K2] and
// [K1,1], or [K1,1] and [1,K2]) and diag(s)(.) is a channel-wise scale.  A convolution with a ternary
// kernel is the ternary matrix product of this library applied to the patches of its input, so the
// two pieces needed are a patch gather and an entry point that runs one ternary stage with its scale.
#include "tsvd_internal.cuh"

namespace {

// out[(n, ho, wo)][(a, b, c)] = x[n, ho*sh + a*dh - ph, wo*sw + b*dw - pw, c]  (zero outside the image)
// one thread per 16-byte-or-smaller run of channels would need alignment rules; this is one thread per
// element, consecutive threads on consecutive channels: reads and writes are coalesced over c.
template <typename T>
__global__ void im2col_nhwc_kernel(const T* __restrict__ x, int n_img, int H, int W, int C, int k1, int k2, int sh, int sw,
                                   int ph, int pw, int dh, int dw, int Ho, int Wo, T* __restrict__ out, long long ld_out)
{
    const long long feat = (long long)k1 * k2 * C;
    const long long total = (long long)n_img * Ho * Wo * feat;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long row = i / feat;
        const int f = (int)(i % feat);
        const int c = f % C, ab = f / C, b = ab % k2, a = ab / k2;
        const int wo = (int)(row % Wo), ho = (int)((row / Wo) % Ho), n = (int)(row / ((long long)Wo * Ho));
        const int h = ho * sh + a * dh - ph, w = wo * sw + b * dw - pw;
        T v = static_cast<T>(0.0f);
        if (h >= 0 && h < H && w >= 0 && w < W) v = x[(((long long)n * H + h) * W + w) * C + c];
        out[row * ld_out + f] = v;
    }
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
    const long long total = (long long)n_img * Ho * Wo * k1 * k2 * C;
    long long blocks = (total + 255) / 256;
    if (blocks > 148LL * 64) blocks = 148LL * 64;
    cudaStream_t st = (cudaStream_t)stream;
    switch (dtype) {
        case TSVD_F32:
            im2col_nhwc_kernel<float><<<(unsigned)blocks, 256, 0, st>>>((const float*)x, n_img, H, W, C, k1, k2, stride_h, stride_w,
                                                                        pad_h, pad_w, dil_h, dil_w, Ho, Wo, (float*)out, ld_out);
            break;
        case TSVD_BF16:
            im2col_nhwc_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, st>>>((const __nv_bfloat16*)x, n_img, H, W, C, k1, k2, stride_h,
                                                                                stride_w, pad_h, pad_w, dil_h, dil_w, Ho, Wo,
                                                                                (__nv_bfloat16*)out, ld_out);
            break;
        case TSVD_I8:
            im2col_nhwc_kernel<int8_t><<<(unsigned)blocks, 256, 0, st>>>((const int8_t*)x, n_img, H, W, C, k1, k2, stride_h, stride_w,
                                                                         pad_h, pad_w, dil_h, dil_w, Ho, Wo, (int8_t*)out, ld_out);
            break;
        default:
            return TSVD_E_DTYPE;
    }
    tsvd_count_launch();
    return cudaGetLastError() == cudaSuccess ? TSVD_OK : TSVD_E_CUDA;
}
