// Ternarisation T(x, theta) of Algorithm 1 (Section "Direct Transition Algorithm to TSVD form"):
// for each vector, the sparsest ternary vector whose angle to it is at most theta.
//
// The optimum keeps sign(x) on the k largest magnitudes for some k, so the search is over k only:
// sort |x| descending, c_k = (sum of the k largest) / sqrt(k) / ||x||, first k with
// c_k >= cos(theta), then keep every entry whose magnitude reaches the k-th largest.
//
// One CTA per vector.  The magnitudes are sorted in shared memory (bitonic network on the next
// power of two, padded with -1 so that the padding sorts last), the prefix sums are taken in
// double precision (a thread sums a contiguous run, the runs are scanned across the block), and the
// first index that reaches the threshold is a block-wide minimum.  The angle test is the only
// place where floating point decides an integer; it is done in double, like the sums, so that it
// agrees with a double-precision evaluation except for cosines within rounding of cos(theta).
#include "tsvd_internal.cuh"

namespace {

constexpr int TERN_THREADS = 1024;

__device__ __forceinline__ double block_sum(double v, double* red)
{
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = (threadIdx.x & 31) < TERN_THREADS / 32 ? red[threadIdx.x & 31] : 0.0;
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    __syncthreads();
    return t;   // the same in every thread
}

// grid: n_vec CTAs of 1024 threads; dynamic shared memory: P floats (P = len rounded up to a power
// of two, at least 2048 so that every thread owns a run of whole elements)
__global__ void __launch_bounds__(TERN_THREADS)
ternarize_kernel(const float* __restrict__ x, int len, int ldx, int P, double cos_theta, int8_t* __restrict__ t, int ldt,
                 int* __restrict__ nnz_out)
{
    extern __shared__ float keys[];
    __shared__ double red[32];
    __shared__ double run_base[TERN_THREADS / 32];
    __shared__ int first_k;
    const int tid = threadIdx.x;
    const float* xv = x + (size_t)blockIdx.x * ldx;
    int8_t* tv = t + (size_t)blockIdx.x * ldt;

    double sq = 0.0;
    for (int i = tid; i < P; i += TERN_THREADS) {
        float a = -1.f;
        if (i < len) {
            a = fabsf(xv[i]);
            sq += (double)a * (double)a;
        }
        keys[i] = a;
    }
    if (tid == 0) first_k = 0x7fffffff;
    const double norm = sqrt(block_sum(sq, red));   // (its barriers also publish keys and first_k)

    // bitonic sort, descending.  Exchanges at distance 32 and more go through shared memory with a
    // block-wide barrier each; the last five of every stage (distance 16 .. 1) stay inside the 32
    // consecutive keys a warp holds per round, so they run in registers with shuffles.
    for (int k = 2; k <= P; k <<= 1) {
        for (int j = k >> 1; j >= 32; j >>= 1) {
            for (int i = tid; i < P; i += TERN_THREADS) {
                const int l = i ^ j;
                if (l > i) {
                    const float a = keys[i], b = keys[l];
                    const bool desc = (i & k) == 0;
                    if (desc ? a < b : a > b) { keys[i] = b; keys[l] = a; }
                }
            }
            __syncthreads();
        }
        for (int i = tid; i < P; i += TERN_THREADS) {       // (P is a multiple of the block: whole warps)
            float a = keys[i];
            const bool desc = (i & k) == 0;
            for (int j = (k >> 1) < 16 ? (k >> 1) : 16; j > 0; j >>= 1) {
                const float b = __shfl_xor_sync(0xffffffffu, a, j);
                const bool lower = (i & j) == 0;             // this lane holds the lower index of the pair
                a = (desc == lower) ? fmaxf(a, b) : fminf(a, b);
            }
            keys[i] = a;
        }
        if (k >= 32) __syncthreads();   // below that a thread only ever touches its own keys
    }
    __syncthreads();

    // prefix sums in double: thread `tid` owns the run [tid * run, tid * run + run)
    const int run = P / TERN_THREADS;
    const int i0 = tid * run;
    double mine = 0.0;
    for (int e = 0; e < run; ++e) {
        const int i = i0 + e;
        if (i < len) mine += (double)keys[i];
    }
    // exclusive scan of the runs' sums: within the warp, then across the warps
    double incl = mine;
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, incl, o);
        if ((tid & 31) >= o) incl += up;
    }
    if ((tid & 31) == 31) run_base[tid >> 5] = incl;
    __syncthreads();
    if (tid < 32) {
        double w = tid < TERN_THREADS / 32 ? run_base[tid] : 0.0, wi = w;
        for (int o = 1; o < 32; o <<= 1) {
            const double up = __shfl_up_sync(0xffffffffu, wi, o);
            if (tid >= o) wi += up;
        }
        if (tid < TERN_THREADS / 32) run_base[tid] = wi - w;   // sum of all earlier warps
    }
    __syncthreads();
    double s = run_base[tid >> 5] + (incl - mine);
    int found = 0x7fffffff;
    if (norm > 0.0) {
        for (int e = 0; e < run; ++e) {
            const int i = i0 + e;
            if (i >= len) break;
            s += (double)keys[i];
            const double c = s / sqrt((double)(i + 1)) / norm;
            if (c >= cos_theta) { found = i; break; }
        }
    }
    if (found != 0x7fffffff) atomicMin(&first_k, found);
    __syncthreads();
    const int ix = first_k;
    if (ix == 0x7fffffff) {   // no ternary vector within the angle: all zeros, count -1
        for (int i = tid; i < len; i += TERN_THREADS) tv[i] = 0;
        if (tid == 0 && nnz_out) nnz_out[blockIdx.x] = -1;
        return;
    }
    const float cut = keys[ix];
    int count = 0;
    for (int i = tid; i < len; i += TERN_THREADS) {
        const float v = xv[i];
        const int8_t tt = fabsf(v) < cut ? (int8_t)0 : (v >= 0.f ? (int8_t)1 : (int8_t)-1);
        tv[i] = tt;
        count += tt != 0;
    }
    if (nnz_out) {
        const double total = block_sum((double)count, red);
        if (tid == 0) nnz_out[blockIdx.x] = (int)total;
    }
}

}  // namespace

extern "C" tsvd_status_t tsvd_ternarize(const float* x, int n_vec, int len, int ldx, double theta, int8_t* t, int ldt,
                                        int* nnz, void* stream)
{
    if (!x || !t) return TSVD_E_NULL;
    if (n_vec < 1 || len < 1 || ldx < len || ldt < len) return TSVD_E_SHAPE;
    if (len > TSVD_TERNARIZE_MAX_LEN) return TSVD_E_TOOBIG;
    if (!(theta >= 0.0) || !(theta <= 1.5707963267948966)) return TSVD_E_SHAPE;
    int P = 2 * TERN_THREADS;
    while (P < len) P <<= 1;
    const size_t smem = (size_t)P * sizeof(float);
    static bool attr_set[64] = {};
    int dev = 0;
    TSVD_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        TSVD_CUDA_OK(cudaFuncSetAttribute(ternarize_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)(TSVD_TERNARIZE_MAX_LEN * sizeof(float))));
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    ternarize_kernel<<<(unsigned)n_vec, TERN_THREADS, smem, (cudaStream_t)stream>>>(x, len, ldx, P, cos(theta), t, ldt, nnz);
    tsvd_count_launch();
    return cudaGetLastError() == cudaSuccess ? TSVD_OK : TSVD_E_CUDA;
}
