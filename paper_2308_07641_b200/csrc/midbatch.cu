// Five to thirty-two tokens: one launch per stage (Table S1 rows "V(.)" with its scale, and "U(.)"),
// the contraction on tcgen05 with the work of a 128-row tile shared by the CTAs of a thread-block cluster.
//
// For so few tokens neither of the other forms fits well: the warp-level MMA of the decode kernels is
// a quarter as fast and at sixteen tokens its instructions, not the packed codes, set the time; the
// tile kernels of the large batches need a launch for each conversion to digits and, to occupy the
// SMs, a contraction split over CTAs whose parts meet through global atomics (four launches).  Here a
// cluster of 4 CTAs takes one tile of 128 rows and splits its contraction: every CTA
//   - expands its slab of the packed codes (at most eight blocks of 128 columns) straight into tensor
//     memory, where the whole slab's A operand fits beside the accumulator (4 warps, thread = row),
//   - converts the same slab of the stage's input into digits in shared memory, a warp per token, with a
//     power-of-two scale per token and slab (never coarser than one scale per token) (16 warps),
//   - contracts them with tcgen05.mma (M = 128, N = digits x tokens <= 256; one thread issues),
//   - and sends its partial results, as float (the exact integers for int8 activations in the V-stage),
//     to the CTA that owns the row through distributed shared memory; after one cluster barrier the
//     owner adds the parts in a fixed order and applies S, or the bias, and the output rounding.
// No global atomics, no scratch besides t = S*(V x); deterministic.  Results agree with the other
// kernel families within the tolerance, not bit for bit (the per-slab scales).
#include "digits.cuh"
#include "sm100_ptx.cuh"
#include "tsvd_internal.cuh"

namespace {

using namespace ptx;

constexpr int MID_THREADS = 672;       // warps 0-3: expand, then epilogue; 4: tensor memory and MMA issue; 5-20: convert
constexpr int MID_CONV_WARPS = 16;
constexpr int MID_MMA_WARP = 4, MID_CONV_WARP0 = 5;
constexpr int MID_MAX_BLOCKS = 8;      // blocks of 128 columns per CTA: 32 tensor-memory columns of A each
constexpr int MID_A_COL0 = 256;        // accumulator: columns 0 .. N-1 (N <= 256); A operand from here
constexpr int MID_TMEM_COLS = 512;
constexpr int MID_DIGIT_BYTES_MAX = 160 * 1024;
// Five to thirty-two tokens (five to eight: only where the decode kernels have no cluster form).  With 64-token
// tiles the digits of a slab of 1024 columns no longer fit shared memory, and clusters of eight CTAs on half the
// slab measured far slower (4096^3 at 48 and 64 tokens: 57 and 64 us against 29 us for 65 tokens on the tile kernels).
constexpr int MID_MAX_B = 32, MID_MIN_B = 5;
constexpr int MID_CL = 4;

enum { MID_STAGE_V = 0, MID_STAGE_U = 1 };

struct MidParams {
    const uint4* units;   // packed ternary operand
    int R, C, C_pad, KB;  // logical rows and columns, padded columns, blocks of 128 columns
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
    const float* bias;    // U-stage, optional (padded to R_pad)
    int* status;
    unsigned long long* stamp;
    int wait_limit;       // bound of the barrier waits in units of 2^20 clocks (0: default)
    int test_stall;       // test hook: the digits are never declared ready, so the waits must give up
    PatchGather pg;       // V-stage: the tokens are patches of the image batch at `in` (C = 0: rows of a matrix)
};

#ifdef TSVD_PHASES   // development builds: finer time stamps from single threads of a middle CTA
#define PH(k, thread) do { if (p.stamp && blockIdx.x == (gridDim.x / 2) && tid == (thread)) p.stamp[2 + (k)] = tsvd_globaltimer(); } while (0)
#else
#define PH(k, thread) do { } while (0)
#endif

__device__ __forceinline__ void st_cluster_b32(uint32_t cluster_addr, uint32_t bits)
{
    asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(cluster_addr), "r"(bits) : "memory");
}

// grid: (R_pad / 128) * CL CTAs in clusters of CL; CTA c of a cluster takes blocks [c KB / CL, (c+1) KB / CL).
// Dynamic shared memory (1024-aligned): digits [blocks][NT rows][128] | packed codes [blocks][4 KiB] | slots [CL][TOK][128 / CL] |
// scale [TOK] | barriers
template <typename IN_T, int ND, int TOK, int STAGE, int CL>
__global__ void __launch_bounds__(MID_THREADS, 1)
ternary_cluster_mma_kernel(const MidParams p)
{
    constexpr bool kInt = sizeof(IN_T) == 1;
    constexpr bool kExact = kInt && STAGE == MID_STAGE_V;   // partial sums travel as integers
    constexpr int NT = ND * TOK;
    constexpr int ROWS_OWN = 128 / CL;
    static_assert(!kInt || ND == 1, "int8 activations are their own digit");
    static_assert(TOK % 16 == 0 && NT <= 256, "tile shape");
    constexpr uint32_t TILE_BYTES = NT * 128;
    constexpr uint32_t IDESC = umma_idesc_s8(128, NT);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t c = cluster_ctarank();
    const int tile = (int)blockIdx.x / CL;
    const int kb0 = (int)c * p.KB / CL, kb1 = ((int)c + 1) * p.KB / CL;
    const int n_blk = kb1 - kb0;                       // 0 .. MID_MAX_BLOCKS (the host checks the upper end)
    const int blk_cap = (p.KB + CL - 1) / CL;          // the most any CTA of the cluster has: same layout in all
    int8_t* digits = reinterpret_cast<int8_t*>(smem);
    uint4* codes = reinterpret_cast<uint4*>(smem + (size_t)blk_cap * TILE_BYTES);        // [blocks][2][128] packed units
    uint32_t* slots = reinterpret_cast<uint32_t*>(codes + (size_t)blk_cap * 256);         // [CL][TOK][ROWS_OWN]
    float* scale = reinterpret_cast<float*>(slots + CL * TOK * ROWS_OWN);
    uint64_t* a_ready = reinterpret_cast<uint64_t*>(scale + TOK);   // [MID_MAX_BLOCKS] block j of A is in tensor memory
    uint64_t* d_ready = a_ready + MID_MAX_BLOCKS;                   // the slab's digits are in shared memory
    uint64_t* done = d_ready + 1;                                   // all MMAs have completed
    uint64_t* c_ready = done + 1;                                   // the slab's packed codes are in shared memory
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(c_ready + 1);
    volatile int* ctl = reinterpret_cast<volatile int*>(tmem_slot + 1);   // [2]: abort flag, wait limit

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int j = 0; j < MID_MAX_BLOCKS; ++j) mbar_init(&a_ready[j], 4);
        mbar_init(d_ready, MID_CONV_WARPS);
        mbar_init(done, 1);
        mbar_init(c_ready, 1);
        ctl[0] = 0;
        ctl[1] = p.wait_limit > 0 ? p.wait_limit : kWaitLimitDefault;
        fence_mbar_init();
    }
    // The slab's packed codes (contiguous: 4 KiB per block) are requested as one bulk copy before anything
    // else -- no kernel writes them -- so that they travel while the kernel before this one still runs.
    if (tid == 0 && n_blk > 0) {
        mbar_arrive_expect_tx(c_ready, (uint32_t)n_blk * 4096u);
        bulk_g2s(codes, p.units + ((size_t)tile * (size_t)(p.C_pad >> 6) + (size_t)(2 * kb0)) * 128, (uint32_t)n_blk * 4096u, c_ready);
    }
    if (warp == MID_MMA_WARP) {
        tmem_alloc(tmem_slot, MID_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // A programmatic dependent of the kernel before it in the stream: the stage's input is read (by the
    // converting warps) and the output written (by everyone, after the cluster barrier) only after that
    // kernel has completed; expanding the codes into tensor memory depends on nothing it does.
    pdl_launch_dependents();

    if (warp < 4) {
        // ---- expanders: thread = row of the tile = tensor-memory lane ----
        const uint32_t a_lane = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)MID_A_COL0;
        bool arrived = n_blk == 0 || mbar_wait(c_ready, 0, ctl);
        for (int j = 0; j < n_blk && arrived; ++j) {
            const uint4 u0 = codes[j * 256 + tid], u1 = codes[j * 256 + 128 + tid];
            uint32_t o[32];   // the row's 128 int8 values of this block, four per 32-bit column
            tsvd_expand16(u0.x, *reinterpret_cast<uint32_t(*)[4]>(&o[0]));
            tsvd_expand16(u0.y, *reinterpret_cast<uint32_t(*)[4]>(&o[4]));
            tsvd_expand16(u0.z, *reinterpret_cast<uint32_t(*)[4]>(&o[8]));
            tsvd_expand16(u0.w, *reinterpret_cast<uint32_t(*)[4]>(&o[12]));
            tsvd_expand16(u1.x, *reinterpret_cast<uint32_t(*)[4]>(&o[16]));
            tsvd_expand16(u1.y, *reinterpret_cast<uint32_t(*)[4]>(&o[20]));
            tsvd_expand16(u1.z, *reinterpret_cast<uint32_t(*)[4]>(&o[24]));
            tsvd_expand16(u1.w, *reinterpret_cast<uint32_t(*)[4]>(&o[28]));
            tmem_st32(a_lane + (uint32_t)(32 * j), o);
            tmem_st_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&a_ready[j]);
        }
    } else if (warp >= MID_CONV_WARP0) {
        // ---- digits of the slab, a warp per token: a lane holds its (up to two) chunks of 16 values
        //      between the maximum and the conversion ----
        pdl_wait();
        if (warp == MID_CONV_WARP0) tsvd_stamp_begin_any(p.stamp);
        PH(0, MID_CONV_WARP0 * 32);
        const IN_T* in = reinterpret_cast<const IN_T*>(p.in);
        const int col0 = kb0 * 128;
        const int n_chunks = n_blk * 8;
        for (int tb = warp - MID_CONV_WARP0; tb < TOK; tb += MID_CONV_WARPS) {
            const bool live = tb < p.B;
            const IN_T* row = in + (size_t)(live ? tb : 0) * p.ld_in;
            const bool vec_ok = (reinterpret_cast<uintptr_t>(row) & 15) == 0;
            int pg_n = 0, pg_ho = 0, pg_wo = 0;   // patches: (image, output row, output column) of this token
            if (p.pg.C && live) {
                pg_wo = tb % p.pg.Wo;
                pg_ho = (tb / p.pg.Wo) % p.pg.Ho;
                pg_n = tb / (p.pg.Wo * p.pg.Ho);
            }
            float keep[2][16];
            float amax = 0.f;
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int ch = lane + 32 * k;
#pragma unroll
                for (int e = 0; e < 16; ++e) keep[k][e] = 0.f;
                if (live && ch < n_chunks) {
                    if (p.pg.C) {   // a chunk lies inside one run of channels, past the row's end, or outside the image
                        const int f0 = col0 + ch * 16;
                        const IN_T* src = f0 < p.pg.feat ? tsvd_patch_ptr<IN_T>(p.pg, in, pg_n, pg_ho, pg_wo, f0) : nullptr;
                        if (src) load16<IN_T>(src, 0, 16, true, keep[k]);
                    } else {
                        load16<IN_T>(row, col0 + ch * 16, p.C, vec_ok, keep[k]);
                    }
#pragma unroll
                    for (int e = 0; e < 16; ++e) amax = fmaxf(amax, fabsf(keep[k][e]));
                }
            }
            float qscale = 1.f;
            PH(1, MID_CONV_WARP0 * 32);
            if constexpr (!kInt) {
                for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
                const int E = tsvd_quant_exponent(amax);
                qscale = tsvd_pow2(8 * ND - 2 - E);
                if (lane == 0) scale[tb] = tsvd_pow2(E - (8 * ND - 2));   // value = q * scale
            } else {
                if (lane == 0) scale[tb] = 1.f;
            }
            unsigned range_cnt = 0;
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int ch = lane + 32 * k;
                if (ch < n_chunks) {
                    uint32_t dig[ND][4];
#pragma unroll
                    for (int d = 0; d < ND; ++d)
#pragma unroll
                        for (int w = 0; w < 4; ++w) dig[d][w] = 0;
                    if (live) {
                        int q[16];
                        if constexpr (!kInt) {   // range diagnostic: one value in four (a slab may be 128 values short)
#pragma unroll
                            for (int e = 0; e < 16; e += 4) tsvd_range_sample(range_cnt, keep[k][e], qscale);
                        }
                        if constexpr (ND <= 3) {
#pragma unroll
                            for (int e = 0; e < 16; ++e) q[e] = tsvd_round_bits(keep[k][e], qscale);
                            digits_of<ND, 4>(q, dig, TSVD_ROUND_BIAS);
                        } else {
#pragma unroll
                            for (int e = 0; e < 16; ++e) q[e] = __float2int_rn(keep[k][e] * qscale);
                            digits_of<ND, 4>(q, dig);
                        }
                    }
                    // K-major 128-byte-swizzle operand layout: row d*TOK + tb of the block's tile, 16-byte
                    // chunk cc at position cc ^ (row & 7)  (TOK is a multiple of 8: row & 7 = tb & 7)
                    const int j = ch >> 3, cc = ch & 7;
                    int8_t* dst = digits + (size_t)j * TILE_BYTES + tb * 128 + ((cc ^ (tb & 7)) << 4);
#pragma unroll
                    for (int d = 0; d < ND; ++d)
                        *reinterpret_cast<uint4*>(dst + d * (TOK * 128)) = make_uint4(dig[d][0], dig[d][1], dig[d][2], dig[d][3]);
                }
            }
            if constexpr (!kInt) {
                if (tsvd_range_flagged(range_cnt) && lane == 0) atomicOr(p.status, TSVD_DEV_RANGE);
            }
        }
        fence_proxy_async_smem();   // the MMAs read these through the async proxy
        __syncwarp();
        if (lane == 0 && !p.test_stall) mbar_arrive(d_ready);
        PH(2, MID_CONV_WARP0 * 32);
    } else {
        // ---- MMA issue: the whole warp walks the blocks, one elected lane issues ----
        bool alive = n_blk == 0 || mbar_wait(d_ready, 0, ctl);
        const uint64_t b_desc0 = umma_desc_k_sw128(smem_u32(digits));
        for (int j = 0; j < n_blk && alive; ++j) {
            if (!mbar_wait(&a_ready[j], 0, ctl)) { alive = false; break; }
            tc_fence_after_sync();
            if (elect_one()) {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    umma_s8_ts(tmem_base, tmem_base + (uint32_t)(MID_A_COL0 + 32 * j + 8 * k),
                               b_desc0 + (uint64_t)(j * (TILE_BYTES >> 4) + k * 2), IDESC, j != 0 || k != 0);
            }
            __syncwarp();
        }
        if (alive && n_blk > 0 && elect_one()) umma_commit(done);
        __syncwarp();
        PH(3, MID_MMA_WARP * 32);
    }

    if (warp < 4) {
        // ---- epilogue: this thread's row of the accumulator -> its share of every token's result, sent to
        //      the CTA that owns the row ----
        const int r = tid;                                    // row of the tile
        const uint32_t owner = (uint32_t)(r / ROWS_OWN);
        const int ro = r % ROWS_OWN;
        const uint32_t my_slots = cluster_map_u32(smem_u32(slots), owner);
        bool have = mbar_wait(d_ready, 0, ctl);               // (the scales are written by then)
        if (have && n_blk > 0) have = mbar_wait(done, 0, ctl);
        else have = false;
        tc_fence_after_sync();
        PH(4, 0);
        const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
#pragma unroll 1
        for (int g = 0; g < TOK / 8; ++g) {
            if (g * 8 >= p.B) break;                          // uniform
            uint32_t acc[ND][8];
#pragma unroll
            for (int d = 0; d < ND; ++d) {
                if (have) tmem_ld8(t_lane + (uint32_t)(d * TOK + g * 8), acc[d]);
                else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[d][i] = 0u;
                }
            }
            if (have) tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int tok = g * 8 + i;
                uint32_t bits;
                if constexpr (kExact) {
                    bits = acc[0][i];
                } else {
                    float f;
                    if constexpr (ND == 1) f = (float)(int)acc[0][i];
                    else if constexpr (ND == 2) f = (float)((int)acc[0][i] + ((int)acc[1][i] << 8));
                    else {
                        const int lo = (int)acc[0][i] + ((int)acc[1][i] << 8);
                        int hi = (int)acc[2][i];
                        if constexpr (ND == 4) hi += (int)acc[3][i] << 8;
                        f = fmaf((float)hi, 65536.f, (float)lo);
                    }
                    bits = __float_as_uint(f * scale[tok]);   // a power of two: exact
                }
                if (tok < p.B) st_cluster_b32(my_slots + (uint32_t)(((c * TOK + tok) * ROWS_OWN + ro) * 4), bits);
            }
        }
    }
    // every CTA's parts have reached their owners
    tc_fence_before_sync();
    cluster_sync_all();
    pdl_wait();
    PH(5, 0);

    // ---- owner: rows c*ROWS_OWN .. of the tile, all tokens ----
    for (int item = tid; item < TOK * ROWS_OWN; item += MID_THREADS) {
        const int tok = item / ROWS_OWN, ro = item % ROWS_OWN;
        if (tok >= p.B) break;
        const int orow = tile * 128 + (int)c * ROWS_OWN + ro;
        float sum = 0.f;
        int isum = 0;
#pragma unroll
        for (int s = 0; s < CL; ++s) {
            const uint32_t v = slots[(s * TOK + tok) * ROWS_OWN + ro];
            if constexpr (kExact) isum += (int)v;
            else sum += __uint_as_float(v);
        }
        if constexpr (kExact) sum = (float)isum;
        if constexpr (STAGE == MID_STAGE_V) {
            // the K multiplications (Table S1); padded rows have S = 0 and no codes
            reinterpret_cast<float*>(p.out)[(size_t)tok * p.ld_out + orow] = p.S[orow] * sum;
            if (p.z_out && orow < p.R) {
                if (p.z_int) reinterpret_cast<int*>(p.z_out)[(size_t)tok * p.z_ld + orow] = kExact ? isum : (int)sum;
                else reinterpret_cast<float*>(p.z_out)[(size_t)tok * p.z_ld + orow] = sum;
            }
        } else if (orow < p.R) {
            const float yv = p.bias ? sum + __ldg(p.bias + orow) : sum;
            if (p.out_bf16) reinterpret_cast<__nv_bfloat16*>(p.out)[(size_t)tok * p.ld_out + orow] = __float2bfloat16_rn(yv);
            else reinterpret_cast<float*>(p.out)[(size_t)tok * p.ld_out + orow] = yv;
        }
    }

    // ---- teardown ----
    __syncthreads();
    if (ctl[0] && tid == 0) atomicOr(p.status, TSVD_DEV_TIMEOUT);
    tsvd_stamp_end(p.stamp);
    if (warp == MID_MMA_WARP) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, MID_TMEM_COLS);
    }
}

// ---- host side ----------------------------------------------------------------------------------
inline int mid_tok(int B) { return B <= 16 ? 16 : 32; }

// cluster size for a stage (0: this form does not serve it): slabs of at most eight blocks whose digits fit
inline int mid_cluster(int KB, int nt)
{
    const int cap = (KB + MID_CL - 1) / MID_CL;
    return cap <= MID_MAX_BLOCKS && (size_t)cap * nt * 128 <= (size_t)MID_DIGIT_BYTES_MAX ? MID_CL : 0;
}

inline size_t mid_smem_bytes(int KB, int nt, int tok, int cl)
{
    const size_t cap = (KB + cl - 1) / cl;
    return 1024 + cap * nt * 128 + cap * 4096 + (size_t)tok * 128 * 4 + (size_t)tok * 4 + (MID_MAX_BLOCKS + 3) * 8 + 16;
}

template <typename IN_T, int ND, int TOK, int STAGE, int CL>
cudaError_t launch_mid_cl(const MidParams& p, int R_pad, cudaStream_t stream)
{
    static bool attr_set[64] = {};   // per instantiation and device
    int dev = 0;
    cudaError_t e0 = cudaGetDevice(&dev);
    if (e0 != cudaSuccess) return e0;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(ternary_cluster_mma_kernel<IN_T, ND, TOK, STAGE, CL>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(R_pad / 128 * CL));
    cfg.blockDim = dim3(MID_THREADS);
    cfg.dynamicSmemBytes = mid_smem_bytes(p.KB, ND * TOK, TOK, CL);
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CL;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, ternary_cluster_mma_kernel<IN_T, ND, TOK, STAGE, CL>, (const MidParams)p);
    tsvd_count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename IN_T, int ND, int STAGE>
cudaError_t launch_mid(const MidParams& p, int R_pad, cudaStream_t stream)
{
    const int tok = mid_tok(p.B);
    if (mid_cluster(p.KB, ND * tok) != MID_CL) return cudaErrorInvalidConfiguration;
    if (tok == 16) return launch_mid_cl<IN_T, ND, 16, STAGE, MID_CL>(p, R_pad, stream);
    return launch_mid_cl<IN_T, ND, 32, STAGE, MID_CL>(p, R_pad, stream);
}

constexpr int ND_T = 4;   // digits of the intermediate t (fp32), as on the other paths
inline int digits_for_x(tsvd_dtype_t dt, bool wide) { return dt == TSVD_I8 ? 1 : (dt == TSVD_BF16 && !wide) ? 3 : 4; }

}  // namespace

bool tsvd_mid_fits(const tsvd_handle_s* h, int B, tsvd_dtype_t dt, bool wide_x)
{
    if (B < MID_MIN_B || B > MID_MAX_B) return false;
    // one round of clusters: with more row tiles than a quarter of the SMs the launch runs in several rounds of
    // about 6 us each, and one padded token tile on the tile kernels is faster (16384 x 4096 x 4096 at 17 and
    // 32 tokens: 42 and 48 us against 30)
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int rows = (h->V.R_pad > h->U.R_pad ? h->V.R_pad : h->U.R_pad) / 128;
    if (rows * MID_CL > sms) return false;
    const int tok = mid_tok(B);
    return mid_cluster(h->V.C_pad / 128, digits_for_x(dt, wide_x) * tok) != 0 && mid_cluster(h->U.C_pad / 128, ND_T * tok) != 0;
}

// scratch: t = S * (V x), [B][R_pad of V] fp32
size_t tsvd_mid_ws_bytes(const tsvd_handle_s* h, int B) { return (size_t)B * h->V.R_pad * sizeof(float); }

tsvd_status_t tsvd_forward_mid(const ForwardArgs& a, void* ws)
{
    tsvd_handle_s* h = a.h;
    float* t = reinterpret_cast<float*>(ws);
    cudaStream_t st = a.stream;
    MidParams p{};
    p.units = h->V.units; p.R = h->K; p.C = h->N; p.C_pad = h->V.C_pad; p.KB = h->V.C_pad / 128;
    p.in = a.x; p.ld_in = a.ldx; p.B = a.B; p.S = h->S;
    p.out = t; p.ld_out = h->V.R_pad;
    p.z_out = a.z_out; p.z_ld = h->K; p.z_int = (a.dtype == TSVD_I8);
    p.status = h->dev_status; p.stamp = h->prof.slot(1);
    if (a.test_stall) { p.wait_limit = 16; p.test_stall = 1; }   // ~8 ms instead of ~2 s
    if (a.gather) p.pg = *a.gather;
    cudaError_t e;
    h->prof.begin(1, st);
    switch (a.dtype) {
        case TSVD_F32: e = launch_mid<float, 4, MID_STAGE_V>(p, h->V.R_pad, st); break;
        case TSVD_BF16:
            e = a.wide_x ? launch_mid<__nv_bfloat16, 4, MID_STAGE_V>(p, h->V.R_pad, st)
                         : launch_mid<__nv_bfloat16, 3, MID_STAGE_V>(p, h->V.R_pad, st);
            break;
        case TSVD_I8: e = launch_mid<int8_t, 1, MID_STAGE_V>(p, h->V.R_pad, st); break;
        default: return TSVD_E_DTYPE;
    }
    h->prof.end(st);
    if (e != cudaSuccess) return TSVD_E_CUDA;
    if (a.v_only) { *a.t_where = t; return TSVD_OK; }

    MidParams q{};
    q.units = h->U.units; q.R = h->M; q.C = h->K; q.C_pad = h->U.C_pad; q.KB = h->U.C_pad / 128;
    q.in = t; q.ld_in = h->V.R_pad; q.B = a.B;
    q.out = a.y; q.ld_out = a.ldy; q.out_bf16 = (a.dtype == TSVD_BF16) && !a.out_f32;
    q.bias = h->bias; q.status = h->dev_status; q.stamp = h->prof.slot(3);
    if (a.test_stall) { q.wait_limit = 16; q.test_stall = 1; }
    h->prof.begin(3, st);
    e = launch_mid<float, ND_T, MID_STAGE_U>(q, h->U.R_pad, st);
    h->prof.end(st);
    return e == cudaSuccess ? TSVD_OK : TSVD_E_CUDA;
}
