// Index-list form for very sparse rows: y = U(diag(S)(V x)) for one to four tokens with U and V
// stored as lists of their nonzeros.
//
// The paper notes that 2 bits per element is a redundant code when U and V are sparse (Section
// "Connection with BNN and What Next").  Here a row of a ternary matrix is the list of its
// nonzero entries, 16 bits each: (column << 1) | (1 if the entry is -1), rows delimited by a
// row-pointer array.  That is 16 r bits per element against 2, so it is the smaller form below a
// nonzero rate r of 1/8, and the forward then does exactly the additions of Table S1: one per
// nonzero and token, none for a zero.
//
// Two launches, one per stage, as on the decode path.  A CTA first writes the stage's input as
// per-token fixed-point integers q = rint(v * 2^(8 ND - 2 - E)) in shared memory (the same rule,
// and therefore the same integers, as the digit paths; they are just not split into digits),
// then each warp takes one row: its lanes walk the row's list, add or subtract q[column] in
// 64-bit integers, and the lanes' sums are added by shuffles.  Every sum is an exact integer; it
// is rounded to fp32 once.
#include "digits.cuh"
#include "tsvd_internal.cuh"

namespace {

constexpr int IDX_THREADS = 512, IDX_WARPS = IDX_THREADS / 32;
constexpr int IDX_ROWS = IDX_WARPS;   // rows per CTA: one per warp
constexpr int IDX_MAX_SMEM = 200 * 1024;

enum { STAGE_V = 0, STAGE_U = 1 };

struct IndexParams {
    const int* row_ptr;        // [R + 1]
    const uint16_t* entries;   // [nnz]: (column << 1) | negative
    int R, C, C_pad;
    const void* in;            // [B][ld_in]: activations (V-stage) or t (U-stage, fp32)
    int ld_in;
    int B;
    const float* S;            // V-stage
    void* out;                 // V-stage: t fp32 [B][ld_out]; U-stage: y [B][ld_out]
    int ld_out;
    int out_bf16;
    void* z_out;               // V-stage, optional: [B][z_ld] int32 (z_int) or fp32
    int z_ld;
    int z_int;
    const float* bias;         // U-stage, optional: added before the output rounding
    int* status;               // device status word (range diagnostic)
    unsigned long long* stamp; // time stamps of this launch, or null
};

// grid: ceil(R / 16) CTAs of 512 threads.  Dynamic shared memory:
//   q [NTOK][C_pad] int32 | scale [NTOK] | per-warp maxima [NTOK][warps]
template <typename IN_T, int ND, int NTOK, int STAGE>
__global__ void __launch_bounds__(IDX_THREADS)
ternary_index_kernel(const IndexParams p)
{
    extern __shared__ __align__(16) uint8_t smem[];
    constexpr bool kInt = sizeof(IN_T) == 1;
    int* q = reinterpret_cast<int*>(smem);
    float* scale = reinterpret_cast<float*>(q + (size_t)NTOK * p.C_pad);
    float* wmax = scale + NTOK;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const IN_T* in = reinterpret_cast<const IN_T*>(p.in);
    const int row = blockIdx.x * IDX_ROWS + warp;
    // the row's extent does not depend on the kernel before this one
    int e0 = 0, e1 = 0;
    if (row < p.R) { e0 = __ldg(p.row_ptr + row); e1 = __ldg(p.row_ptr + row + 1); }
    // a programmatic dependent of the kernel before it in the stream: the stage's input is read,
    // and its output written, only after this wait
    pdl_wait();
    pdl_launch_dependents();
    tsvd_stamp_begin(p.stamp);

    // ---- the stage's input as fixed-point integers ----
    const int n_chunks = p.C_pad >> 3;
    float qscale[NTOK];
    const IN_T* rows[NTOK];
    bool vec_ok[NTOK];
#pragma unroll
    for (int b = 0; b < NTOK; ++b) {
        qscale[b] = 1.f;
        rows[b] = in + (size_t)(b < p.B ? b : 0) * p.ld_in;   // tokens beyond the batch re-read token 0, unused
        vec_ok[b] = ((reinterpret_cast<uintptr_t>(rows[b])) & 15) == 0;
    }
    if constexpr (!kInt) {
        float amax[NTOK];
#pragma unroll
        for (int b = 0; b < NTOK; ++b) amax[b] = 0.f;
        for (int ch = tid; ch < n_chunks; ch += IDX_THREADS) {
            float v[NTOK][8];
#pragma unroll
            for (int b = 0; b < NTOK; ++b) load8<IN_T>(rows[b], ch * 8, p.C, vec_ok[b], v[b]);
#pragma unroll
            for (int b = 0; b < NTOK; ++b)
#pragma unroll
                for (int e = 0; e < 8; ++e) amax[b] = fmaxf(amax[b], fabsf(v[b][e]));
        }
#pragma unroll
        for (int b = 0; b < NTOK; ++b) {
            for (int o = 16; o > 0; o >>= 1) amax[b] = fmaxf(amax[b], __shfl_xor_sync(0xffffffffu, amax[b], o));
            if (lane == 0) wmax[b * IDX_WARPS + warp] = amax[b];
        }
        __syncthreads();
#pragma unroll
        for (int b = 0; b < NTOK; ++b) {
            float m = wmax[b * IDX_WARPS + (lane & (IDX_WARPS - 1))];
            for (int o = IDX_WARPS / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            const int E = tsvd_quant_exponent(m);
            qscale[b] = tsvd_pow2(8 * ND - 2 - E);
            if (tid == 0) scale[b] = tsvd_pow2(E - (8 * ND - 2));   // value = q * scale
        }
    } else {
        if (tid < NTOK) scale[tid] = 1.f;
    }
    unsigned range_cnt[NTOK];   // range diagnostic: the first value of every chunk is sampled
#pragma unroll
    for (int b = 0; b < NTOK; ++b) range_cnt[b] = 0;
    for (int ch = tid; ch < n_chunks; ch += IDX_THREADS) {
        float v[NTOK][8];
#pragma unroll
        for (int b = 0; b < NTOK; ++b) load8<IN_T>(rows[b], ch * 8, p.C, vec_ok[b], v[b]);
#pragma unroll
        for (int b = 0; b < NTOK; ++b) {
            int qv[8];
            if constexpr (!kInt) { if (b < p.B) tsvd_range_sample(range_cnt[b], v[b][0], qscale[b]); }
#pragma unroll
            for (int e = 0; e < 8; ++e) qv[e] = b < p.B ? __float2int_rn(v[b][e] * qscale[b]) : 0;
            int4* dst = reinterpret_cast<int4*>(q + (size_t)b * p.C_pad + ch * 8);
            dst[0] = make_int4(qv[0], qv[1], qv[2], qv[3]);
            dst[1] = make_int4(qv[4], qv[5], qv[6], qv[7]);
        }
    }
    if constexpr (!kInt) {
#pragma unroll
        for (int b = 0; b < NTOK; ++b)
            if (tsvd_range_flagged(range_cnt[b]) && lane == 0) atomicOr(p.status, TSVD_DEV_RANGE);
    }
    __syncthreads();

    // ---- one row per warp: the additions and subtractions at its nonzeros ----
    long long acc[NTOK];
#pragma unroll
    for (int b = 0; b < NTOK; ++b) acc[b] = 0;
    for (int e = e0 + lane; e < e1; e += 32) {
        const uint32_t ent = __ldg(p.entries + e);
        const int col = (int)(ent >> 1);
        const bool neg = ent & 1u;
#pragma unroll
        for (int b = 0; b < NTOK; ++b) {
            const int v = q[(size_t)b * p.C_pad + col];
            acc[b] += neg ? -(long long)v : (long long)v;
        }
    }
#pragma unroll
    for (int b = 0; b < NTOK; ++b)
        for (int o = 16; o > 0; o >>= 1) acc[b] += __shfl_xor_sync(0xffffffffu, acc[b], o);

    if (row < p.R && lane < NTOK && lane < p.B) {
        long long a = 0;
#pragma unroll
        for (int b = 0; b < NTOK; ++b)
            if (b == lane) a = acc[b];
        const int b = lane;
        const float val = __ll2float_rn(a) * scale[b];   // one rounding; the scale is a power of two
        if constexpr (STAGE == STAGE_V) {
            reinterpret_cast<float*>(p.out)[(size_t)b * p.ld_out + row] = p.S[row] * val;   // the K multiplications
            if (p.z_out) {
                if (p.z_int) reinterpret_cast<int*>(p.z_out)[(size_t)b * p.z_ld + row] = (int)a;
                else reinterpret_cast<float*>(p.z_out)[(size_t)b * p.z_ld + row] = val;
            }
        } else {
            const float yv = p.bias ? val + __ldg(p.bias + row) : val;
            if (p.out_bf16)
                reinterpret_cast<__nv_bfloat16*>(p.out)[(size_t)b * p.ld_out + row] = __float2bfloat16_rn(yv);
            else
                reinterpret_cast<float*>(p.out)[(size_t)b * p.ld_out + row] = yv;
        }
    }
    tsvd_stamp_end(p.stamp);
}

size_t index_smem_bytes(int ntok, int C_pad)
{
    return (size_t)ntok * C_pad * sizeof(int) + (size_t)ntok * sizeof(float) + (size_t)IDX_WARPS * ntok * sizeof(float);
}

template <typename IN_T, int ND, int NTOK, int STAGE>
cudaError_t launch_index(const IndexParams& p, cudaStream_t stream)
{
    static bool attr_set[64] = {};   // per instantiation and device
    const size_t smem = index_smem_bytes(NTOK, p.C_pad);
    int dev = 0;
    cudaError_t e0 = cudaGetDevice(&dev);
    if (e0 != cudaSuccess) return e0;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(ternary_index_kernel<IN_T, ND, NTOK, STAGE>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, IDX_MAX_SMEM);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    PdlLaunch cfg((unsigned)((p.R + IDX_ROWS - 1) / IDX_ROWS), (unsigned)IDX_THREADS, smem, stream);
    const cudaError_t e = cudaLaunchKernelEx(&cfg.cfg, ternary_index_kernel<IN_T, ND, NTOK, STAGE>, (const IndexParams)p);
    tsvd_count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename IN_T, int ND, int STAGE>
cudaError_t launch_index_tokens(const IndexParams& p, cudaStream_t stream)
{
    if (p.B == 1) return launch_index<IN_T, ND, 1, STAGE>(p, stream);
    if (p.B == 2) return launch_index<IN_T, ND, 2, STAGE>(p, stream);
    return launch_index<IN_T, ND, 4, STAGE>(p, stream);
}

constexpr int ND_T = 4;   // the intermediate t (fp32) is quantised as on the digit paths

}  // namespace

// Host side of tsvd_pack with TSVD_PACK_INDEX_LISTS: the nonzeros of a row-major int8 ternary
// matrix as 16-bit entries.  Values were validated by the 2-bit packer before this is called.
tsvd_status_t tsvd_build_index_lists(const int8_t* host, int R, int C, IndexMat* out)
{
    if (C > TSVD_INDEX_MAX_COLUMNS) return TSVD_E_TOOBIG;
    std::vector<int> row_ptr((size_t)R + 1, 0);
    std::vector<uint16_t> entries;
    try {
        entries.reserve((size_t)R * (size_t)C / 4 + 16);
        for (int r = 0; r < R; ++r) {
            const int8_t* src = host + (size_t)r * C;
            for (int c = 0; c < C; ++c)
                if (src[c] != 0) entries.push_back((uint16_t)((c << 1) | (src[c] < 0 ? 1 : 0)));
            if (entries.size() > (size_t)0x7fffffff) return TSVD_E_TOOBIG;
            row_ptr[(size_t)r + 1] = (int)entries.size();
        }
    } catch (const std::bad_alloc&) {
        return TSVD_E_NOMEM;
    }
    out->R = R; out->C = C; out->C_pad = (C + 127) / 128 * 128;
    out->nnz = entries.size();
    if (cudaMalloc(&out->row_ptr, row_ptr.size() * sizeof(int)) != cudaSuccess) { (void)cudaGetLastError(); return TSVD_E_NOMEM; }
    if (cudaMalloc(&out->entries, (entries.size() + 8) * sizeof(uint16_t)) != cudaSuccess) { (void)cudaGetLastError(); return TSVD_E_NOMEM; }
    TSVD_CUDA_OK(cudaMemcpy(out->row_ptr, row_ptr.data(), row_ptr.size() * sizeof(int), cudaMemcpyHostToDevice));
    if (!entries.empty())
        TSVD_CUDA_OK(cudaMemcpy(out->entries, entries.data(), entries.size() * sizeof(uint16_t), cudaMemcpyHostToDevice));
    return TSVD_OK;
}

bool tsvd_index_fits(const tsvd_handle_s* h, int B)
{
    if (!h->Vi.row_ptr || !h->Ui.row_ptr || B < 1 || B > TSVD_INDEX_MAX_B) return false;
    const int ntok = B == 3 ? 4 : B;
    return index_smem_bytes(ntok, h->Vi.C_pad) <= (size_t)IDX_MAX_SMEM &&
           index_smem_bytes(ntok, h->Ui.C_pad) <= (size_t)IDX_MAX_SMEM;
}

tsvd_status_t tsvd_forward_index(const ForwardArgs& a, void* ws)
{
    tsvd_handle_s* h = a.h;
    cudaStream_t st = a.stream;
    float* t = reinterpret_cast<float*>(ws);

    IndexParams p{};
    p.row_ptr = h->Vi.row_ptr; p.entries = h->Vi.entries; p.R = h->K; p.C = h->N; p.C_pad = h->Vi.C_pad;
    p.in = a.x; p.ld_in = a.ldx; p.B = a.B; p.S = h->S;
    p.out = t; p.ld_out = h->V.R_pad;
    p.z_out = a.z_out; p.z_ld = h->K; p.z_int = (a.dtype == TSVD_I8);
    p.status = h->dev_status; p.stamp = h->prof.slot(1);
    cudaError_t e;
    h->prof.begin(1, st);
    switch (a.dtype) {
        case TSVD_F32: e = launch_index_tokens<float, 4, STAGE_V>(p, st); break;
        case TSVD_BF16:
            e = a.wide_x ? launch_index_tokens<__nv_bfloat16, 4, STAGE_V>(p, st) : launch_index_tokens<__nv_bfloat16, 3, STAGE_V>(p, st);
            break;
        case TSVD_I8: e = launch_index_tokens<int8_t, 1, STAGE_V>(p, st); break;
        default: return TSVD_E_DTYPE;
    }
    h->prof.end(st);
    if (e != cudaSuccess) return TSVD_E_CUDA;

    IndexParams u{};
    u.row_ptr = h->Ui.row_ptr; u.entries = h->Ui.entries; u.R = h->M; u.C = h->K; u.C_pad = h->Ui.C_pad;
    u.in = t; u.ld_in = h->V.R_pad; u.B = a.B;
    u.out = a.y; u.ld_out = a.ldy;
    u.out_bf16 = (a.dtype == TSVD_BF16) && !a.out_f32;
    u.bias = h->bias; u.status = h->dev_status; u.stamp = h->prof.slot(3);
    h->prof.begin(3, st);
    e = launch_index_tokens<float, ND_T, STAGE_U>(u, st);
    h->prof.end(st);
    return e == cudaSuccess ? TSVD_OK : TSVD_E_CUDA;
}
