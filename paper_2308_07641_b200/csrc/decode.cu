// Decode path: y = U(diag(S)(V x)) for one to sixteen tokens, bound by streaming the packed codes (a single-CTA
// kernel per 32 rows, described first; from three tokens on a cluster form, described where it is defined).
//
// For so few tokens a 128-row tcgen05 tile is almost empty, and what matters is that every SM
// streams its share of the 2-bit codes (the whole of U and V is read once per forward) with as
// little fixed cost and as few instructions per code as possible.  Two launches, one per stage
// (Table S1 rows "V(.)" and "U(.)"): each CTA first turns the stage's input (x, or t = S*(V x))
// into the same per-token fixed-point digits as the tensor-core path, in shared memory, then
// takes 32 rows of the packed matrix.  The additions run on the warp-level integer MMA
// (m16n8k32, int8 x int8 -> int32, operands in registers): the A operand is 16 rows x 32 columns
// of codes expanded to int8 in registers (two byte permutes per eight entries), the B operand 32
// columns x 8 (token, digit) pairs read from shared memory, so one instruction does the work of
// 128 four-way dot products and the instruction count per code is set by the expansion alone
// (9 per 16 entries).  A per-lane dot-product kernel issued four dot products per 16 entries,
// token and digit on top of that: 1.8 us per token and stage on a 4096 x 4096 matrix against
// 0.65 us to stream it.  All sums are
// exact integers, so the result does not depend on how the columns are split over the warps.
//
// Column order inside an MMA: a thread (row group g = lane / 4, quarter q = lane % 4) loads word q
// of the 16-byte unit of rows g and g + 8, i.e. columns 16q .. 16q+15 of a 64-column group, and
// one 16-byte slice of digits for the same columns.  The instruction's contraction index is
// only a label, so the first MMA of a group takes columns 16q .. 16q+7 of every quarter and the
// second 16q+8 .. 16q+15; each loaded word and digit slice is used whole and nothing is shuffled.
#include "digits.cuh"
#include "tsvd_internal.cuh"

namespace {

constexpr int GEMV_THREADS = 512, GEMV_WARPS = GEMV_THREADS / 32;
constexpr int GEMV_ROWS = 32;       // rows per CTA: two MMA row tiles
constexpr int GEMV_PRE = 4;         // column groups a warp has in flight at a time
constexpr int GEMV_DIG_PAD = 64;    // bytes between digit rows beyond C_pad: eight rows x four quarters hit all banks
constexpr int GEMV_MAX_SMEM = 224 * 1024;

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
    const float* bias;    // U-stage, optional (padded to R_pad): added before the output rounding
    int* status;          // device status word (range diagnostic)
    unsigned long long* stamp;   // time stamps of this launch, or null
};

// D (16 x 8, int32) += A (16 x 32, int8, rows) * B (32 x 8, int8, columns).  Lane (g, q):
// a0/a2 = row g, contraction bytes 4q..4q+3 and 16+4q..; a1/a3 = row g + 8, the same bytes;
// b0/b1 = column g, the same bytes; c0,c1 = row g, columns 2q, 2q+1; c2,c3 = row g + 8.
__device__ __forceinline__ void mma_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// A streaming 32-bit load that stays where it is written: the compiler moves an ordinary load
// down to its first use, which for the codes is after the digit conversion, and their trip from
// HBM (the longest wait of the kernel) would then start only there.
__device__ __forceinline__ uint32_t ld_stream_now(const uint32_t* ptr)
{
    uint32_t v;
    asm volatile("ld.global.cs.b32 %0, [%1];" : "=r"(v) : "l"(ptr));
    return v;
}

// grid: R_pad / 32 CTAs of 512 threads.  Dynamic shared memory:
//   digits [NTOK*ND][C_pad + 64] int8 | sums [NTOK*ND][32 rows] int32 |
//   scale [NTOK] | per-warp maxima [NTOK][warps]
// Registers: at one token the kernel stays within 64 per thread, so that two CTAs fit an SM: that
// is what lets the next kernel's CTAs start, and request their codes, while this kernel still runs
// (a variant that needed 67 took 7.9 instead of 6.2 us per forward).  With more tokens the
// conversion's working set does not fit 64 registers (capped, it spilled: 16.6 and 22 us at four
// tokens against 9.6), so those run one CTA per SM.
template <typename IN_T, int ND, int NTOK, int STAGE>
__global__ void __launch_bounds__(GEMV_THREADS, NTOK == 1 ? 2 : 1)
ternary_gemv_kernel(const GemvParams p)
{
    extern __shared__ __align__(16) uint8_t smem[];
    constexpr bool kInt = sizeof(IN_T) == 1;
    static_assert(!kInt || ND == 1, "int8 activations are their own digit");
    constexpr int NCOL = NTOK * ND;            // (token, digit) pairs = columns of the B operand
    constexpr int NT = (NCOL + 7) / 8;         // MMA column tiles
    const int dstride = p.C_pad + GEMV_DIG_PAD;
    int8_t* dig = reinterpret_cast<int8_t*>(smem);
    int* red = reinterpret_cast<int*>(smem + (size_t)NCOL * dstride);
    float* scale = reinterpret_cast<float*>(red + NCOL * GEMV_ROWS);
    float* wmax = scale + NTOK;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, q = lane & 3;
    const IN_T* in = reinterpret_cast<const IN_T*>(p.in);
    for (int i = tid; i < NCOL * GEMV_ROWS; i += GEMV_THREADS) red[i] = 0;   // the warps add into these after two barriers

    // Warp w takes column groups w, w + 16, ..; a lane's word of rows 16h + g and 16h + g + 8
    // (h = 0, 1) of each.  One warp-wide load is 8 rows x 16 bytes = 128 contiguous bytes.  The
    // first GEMV_PRE groups are requested before anything else, so that their trip from HBM
    // overlaps with the digit conversion below.  All addresses are one pointer plus constants:
    // the 32 rows lie in one 128-row block, and 16 column groups on is 16 blocks of 2 KiB on.
    // (The kernel is bound by the number of instructions it issues, not by any one wait: address
    // arithmetic repeated per load was a third of them.)
    const int n_groups = p.C_pad >> 6;
    constexpr int GROUP_STEP = GEMV_WARPS * 128 * 4;   // words between a warp's consecutive column groups
    const uint32_t* wp = reinterpret_cast<const uint32_t*>(p.units) +
                         (tsvd_unit_index(blockIdx.x * GEMV_ROWS, warp, p.C_pad) + g) * 4 + q;
    uint32_t w[GEMV_PRE][2][2];
#pragma unroll
    for (int i = 0; i < GEMV_PRE; ++i) {
        const bool there = warp + i * GEMV_WARPS < n_groups;
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int r = 0; r < 2; ++r)
                w[i][h][r] = there ? ld_stream_now(wp + i * GROUP_STEP + (16 * h + 8 * r) * 4) : 0u;
    }
    // Both stages are launched as programmatic dependents of the kernel before them in the
    // stream: their CTAs may start, and request their first codes (which no kernel writes), while
    // that kernel still runs.  The stage's input (x, or t from the V-stage) is complete and
    // visible only after this wait, and the stage's output is written after it, so a kernel that
    // still reads t or y is never overtaken.  The next kernel in the stream may start likewise.
    pdl_wait();
    pdl_launch_dependents();
    tsvd_stamp_begin(p.stamp);

    // ---- the stage's input as fixed-point digits (every CTA makes its own copy).  A thread takes
    //      chunks of 8 consecutive columns; all loads of a pass are independent, so a pass costs
    //      about one trip to L2, and the first chunk of each token stays in registers between the
    //      maximum pass and the conversion pass ----
    // Up to four tokens are converted at a time (eight tokens: two such passes, whose working set
    // still fits the registers).
    const int n_chunks = p.C_pad >> 3;
    constexpr int TB = NTOK < 4 ? NTOK : 4;
#pragma unroll
    for (int b0 = 0; b0 < NTOK; b0 += TB) {
        float keep[TB][8];
        float qscale[TB];
    #pragma unroll
        for (int b = 0; b < TB; ++b) qscale[b] = 1.f;
        // tokens beyond the batch re-read token 0 (the loads of all tokens are then unconditional and go
        // out together); what they read is never used
        const IN_T* rows[TB];
        bool vec_ok[TB];
    #pragma unroll
        for (int b = 0; b < TB; ++b) {
            rows[b] = in + (size_t)(b0 + b < p.B ? b0 + b : 0) * p.ld_in;
            vec_ok[b] = ((reinterpret_cast<uintptr_t>(rows[b])) & 15) == 0;
        }
        bool all_vec = true;   // every token's row allows vector loads: one test per chunk, and the loads in a row
    #pragma unroll
        for (int b = 0; b < TB; ++b) all_vec = all_vec && vec_ok[b];
        auto load_tokens = [&](int ch, float (&v)[TB][8]) {
            if (all_vec && ch * 8 + 8 <= p.C) {
    #pragma unroll
                for (int b = 0; b < TB; ++b) load8<IN_T>(rows[b], ch * 8, 0x7fffffff, true, v[b]);
            } else {
    #pragma unroll
                for (int b = 0; b < TB; ++b) load8<IN_T>(rows[b], ch * 8, p.C, vec_ok[b], v[b]);
            }
        };
        if constexpr (!kInt) {
            float amax[TB];
    #pragma unroll
            for (int b = 0; b < TB; ++b) amax[b] = 0.f;
            for (int ch = tid; ch < n_chunks; ch += GEMV_THREADS) {
                float v[TB][8];
                load_tokens(ch, v);
    #pragma unroll
                for (int b = 0; b < TB; ++b) {
    #pragma unroll
                    for (int e = 0; e < 8; ++e) amax[b] = fmaxf(amax[b], fabsf(v[b][e]));
                    if (ch == tid) {
    #pragma unroll
                        for (int e = 0; e < 8; ++e) keep[b][e] = v[b][e];
                    }
                }
            }
    #pragma unroll
            for (int b = 0; b < TB; ++b) {
                for (int o = 16; o > 0; o >>= 1) amax[b] = fmaxf(amax[b], __shfl_xor_sync(0xffffffffu, amax[b], o));
                if (lane == 0) wmax[(b0 + b) * GEMV_WARPS + warp] = amax[b];
            }
            __syncthreads();
    #pragma unroll
            for (int b = 0; b < TB; ++b) {
                // the sixteen warps' maxima: one per lane of each half-warp, then across its lanes
                float m = wmax[(b0 + b) * GEMV_WARPS + (lane & (GEMV_WARPS - 1))];
                for (int o = GEMV_WARPS / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
                const int E = tsvd_quant_exponent(m);
                qscale[b] = tsvd_pow2(8 * ND - 2 - E);
                if (tid == 0) scale[b0 + b] = tsvd_pow2(E - (8 * ND - 2));   // value = q * scale
            }
        } else {
            if (tid < NTOK) scale[tid] = 1.f;
        }
        unsigned range_cnt[TB];   // range diagnostic: the first value of every chunk is sampled
    #pragma unroll
        for (int b = 0; b < TB; ++b) range_cnt[b] = 0;
        for (int ch = tid; ch < n_chunks; ch += GEMV_THREADS) {
            float v[TB][8];
            if (!kInt && ch == tid) {
    #pragma unroll
                for (int b = 0; b < TB; ++b)
    #pragma unroll
                    for (int e = 0; e < 8; ++e) v[b][e] = keep[b][e];
            } else {
                load_tokens(ch, v);
            }
    #pragma unroll
            for (int b = 0; b < TB; ++b) {
                uint32_t dw[ND][2];
    #pragma unroll
                for (int d = 0; d < ND; ++d) dw[d][0] = dw[d][1] = 0u;
                if (b0 + b < p.B) {
                    int qv[8];
                    if constexpr (!kInt) tsvd_range_sample(range_cnt[b], v[b][0], qscale[b]);
                    if constexpr (ND <= 3) {   // |q| <= 2^22: round by adding a constant, whose image the digit offset absorbs
    #pragma unroll
                        for (int e = 0; e < 8; ++e) qv[e] = tsvd_round_bits(v[b][e], qscale[b]);
                        digits_of<ND, 2>(qv, dw, TSVD_ROUND_BIAS);
                    } else {
    #pragma unroll
                        for (int e = 0; e < 8; ++e) qv[e] = __float2int_rn(v[b][e] * qscale[b]);
                        digits_of<ND, 2>(qv, dw);
                    }
                }
    #pragma unroll
                for (int d = 0; d < ND; ++d)
                    *reinterpret_cast<uint2*>(dig + (size_t)((b0 + b) * ND + d) * dstride + ch * 8) = make_uint2(dw[d][0], dw[d][1]);
            }
        }
        if constexpr (!kInt) {
    #pragma unroll
            for (int b = 0; b < TB; ++b)
                if (tsvd_range_flagged(range_cnt[b]) && lane == 0) atomicOr(p.status, TSVD_DEV_RANGE);
        }
    }
    __syncthreads();

    // ---- stream the codes ----
    int acc[2][NT][4];
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[h][j][c] = 0;

    const int8_t* dp = dig + (size_t)g * dstride + warp * 64 + q * 16;   // this lane's digit slice of group `warp`
    bool col_there[NT];
#pragma unroll
    for (int j = 0; j < NT; ++j) col_there[j] = 8 * j + g < NCOL;
#pragma unroll 1
    for (int first = warp; first < n_groups; first += GEMV_PRE * GEMV_WARPS) {
        wp += GEMV_PRE * GROUP_STEP;
        uint32_t wn[GEMV_PRE][2][2];   // the next groups, in flight while these are summed
#pragma unroll
        for (int i = 0; i < GEMV_PRE; ++i)
#pragma unroll
            for (int h = 0; h < 2; ++h) wn[i][h][0] = wn[i][h][1] = 0u;
        if (first + GEMV_PRE * GEMV_WARPS < n_groups) {   // one test when nothing is left (the usual case at 4096 columns)
#pragma unroll
            for (int i = 0; i < GEMV_PRE; ++i) {
                if (first + (GEMV_PRE + i) * GEMV_WARPS < n_groups) {
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int r = 0; r < 2; ++r)
                            wn[i][h][r] = ld_stream_now(wp + i * GROUP_STEP + (16 * h + 8 * r) * 4);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < GEMV_PRE; ++i) {
            if (first + i * GEMV_WARPS < n_groups) {   // the same for the whole warp
                uint4 xd[NT];      // digits of columns 16q .. 16q+15 of this group, (token, digit) pair 8j + g
#pragma unroll
                for (int j = 0; j < NT; ++j)
                    xd[j] = col_there[j] ? *reinterpret_cast<const uint4*>(dp + (size_t)(8 * j) * dstride + i * GEMV_WARPS * 64)
                                         : make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t e0[4], e1[4];   // sixteen entries of rows 16h + g and 16h + g + 8 as int8
                    tsvd_expand16(w[i][h][0], e0);
                    tsvd_expand16(w[i][h][1], e1);
#pragma unroll
                    for (int j = 0; j < NT; ++j) {
                        mma_s8(acc[h][j], e0[0], e1[0], e0[1], e1[1], xd[j].x, xd[j].y);
                        mma_s8(acc[h][j], e0[2], e1[2], e0[3], e1[3], xd[j].z, xd[j].w);
                    }
                }
            }
        }
        dp += GEMV_PRE * GEMV_WARPS * 64;
#pragma unroll
        for (int i = 0; i < GEMV_PRE; ++i)
#pragma unroll
            for (int h = 0; h < 2; ++h) { w[i][h][0] = wn[i][h][0]; w[i][h][1] = wn[i][h][1]; }
    }

    // ---- the warps took different column groups: their sums meet in shared memory (integer
    //      additions: exact in any order) ----
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int n = 8 * j + 2 * q + (c & 1), r = 16 * h + g + 8 * (c >> 1);
                if (n < NCOL) atomicAdd(&red[n * GEMV_ROWS + r], acc[h][j][c]);
            }
    __syncthreads();

    // ---- thread (token, row): digits -> fp32 -> the stage's output ----
    if (tid < NTOK * GEMV_ROWS) {
        const int b = tid / GEMV_ROWS, r = tid % GEMV_ROWS;
        const int orow = blockIdx.x * GEMV_ROWS + r;
        if (b < p.B) {
            int a[ND];
#pragma unroll
            for (int d = 0; d < ND; ++d) a[d] = red[(b * ND + d) * GEMV_ROWS + r];
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
                const float yv = p.bias ? val + __ldg(p.bias + orow) : val;
                if (p.out_bf16)
                    reinterpret_cast<__nv_bfloat16*>(p.out)[(size_t)b * p.ld_out + orow] = __float2bfloat16_rn(yv);
                else
                    reinterpret_cast<float*>(p.out)[(size_t)b * p.ld_out + orow] = yv;
            }
        }
    }
    tsvd_stamp_end(p.stamp);
}

#ifdef TSVD_PHASES   // development builds: finer time stamps from one warp of a middle CTA
#define PH(k) do { if (p.stamp && blockIdx.x == (gridDim.x / 2) && tid == 96) p.stamp[2 + (k)] = tsvd_globaltimer(); } while (0)
#else
#define PH(k) do { } while (0)
#endif

// ---------------------------------------------------------------------------------------
// Cluster form of the same stage, for contractions of 1024 columns and more.  In the kernel
// above every CTA reads and converts the whole stage input; at four tokens that takes longer than
// streaming the CTA's codes.  Here four CTAs of a thread-block cluster share a tile of 128 rows
// and split its CONTRACTION: each reads and converts only its quarter of the columns (with its
// own power-of-two scale per token: a finer scale than one per token, never a coarser one),
// contracts all 128 rows against that quarter, and the four partial results meet through
// distributed shared memory: CTA c of the cluster finishes rows 32c .. 32c+31, every CTA stores
// its partial sums of those rows into a slot of CTA c's shared memory, one cluster barrier, and
// the owner adds the four slots in a fixed order (deterministic; for int8 activations the slots
// hold the exact integers).  No global atomics, no second pass over the input.
// ---------------------------------------------------------------------------------------
constexpr int CLUSTER_CTAS = 4;
constexpr int CLUSTER_ROWS = 128;           // rows of a cluster's tile = rows every CTA of it contracts
constexpr int CLUSTER_OWN = CLUSTER_ROWS / CLUSTER_CTAS;   // rows a CTA finishes
constexpr int CLUSTER_MIN_GROUPS = 16;      // use this form from 1024 columns on
constexpr int CLUSTER_MIN_TOKENS = 3;        // and from three tokens on

__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// address of `local` (a shared-memory address of this CTA) in the shared memory of CTA `rank` of the cluster
__device__ __forceinline__ uint32_t cluster_map(const void* local, uint32_t rank)
{
    uint32_t a = static_cast<uint32_t>(__cvta_generic_to_shared(local)), r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_store(uint32_t remote, uint32_t bits)
{
    asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(remote), "r"(bits) : "memory");
}
__device__ __forceinline__ void cluster_barrier()
{
    asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}

__host__ __device__ inline int cluster_slab_groups(int C_pad) { return ((C_pad >> 6) + CLUSTER_CTAS - 1) / CLUSTER_CTAS; }

// grid: (R_pad / 128) * 4 CTAs of 512 threads in clusters of 4.  Dynamic shared memory:
//   digits [NTOK*ND][slab + 64] int8 | sums [4 column parts][NTOK*ND][128] int32 | slots [4][NTOK][32] | scale [NTOK] |
//   max bits [NTOK] | range counts [NTOK]
// Warp w: rows 32 (w % 4) .. +31 of the tile (two MMA row tiles), column part w / 4 of the CTA's slab:
// per round of 16 groups it takes groups 4 (w / 4) .. +3.
template <typename IN_T, int ND, int NTOK, int STAGE>
__global__ void __launch_bounds__(GEMV_THREADS, NTOK <= 2 ? 2 : 1)
ternary_gemv_cluster_kernel(const GemvParams p)
{
    extern __shared__ __align__(16) uint8_t smem[];
    constexpr bool kInt = sizeof(IN_T) == 1;
    constexpr bool kIntSlots = kInt && STAGE == STAGE_V;   // exact integer partial sums
    constexpr int NCOL = NTOK * ND;
    constexpr int NT = (NCOL + 7) / 8;
    const int n_groups = p.C_pad >> 6;
    const int gq = cluster_slab_groups(p.C_pad);
    const uint32_t rank = cluster_rank();
    const int g0 = (int)rank * gq, g1 = min(n_groups, g0 + gq);      // this CTA's column groups
    const int dstride = gq * 64 + GEMV_DIG_PAD;
    int8_t* dig = reinterpret_cast<int8_t*>(smem);
    int* red = reinterpret_cast<int*>(smem + (size_t)NCOL * dstride);
    uint32_t* slots = reinterpret_cast<uint32_t*>(red + 4 * NCOL * CLUSTER_ROWS);   // [4][NTOK][32]
    float* scale = reinterpret_cast<float*>(slots + CLUSTER_CTAS * NTOK * CLUSTER_OWN);
    unsigned* smax = reinterpret_cast<unsigned*>(scale + NTOK);
    unsigned* srange = smax + NTOK;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, q = lane & 3;
    const int rp = warp & 3, cp = warp >> 2;
    const int tile = blockIdx.x / CLUSTER_CTAS;
    const IN_T* in = reinterpret_cast<const IN_T*>(p.in);
    if (tid < NTOK) { smax[tid] = 0u; srange[tid] = 0u; }

    // this lane's codes of the first round, requested before the wait (they travel from HBM meanwhile)
    constexpr int GROUP_WORDS = 128 * 4;
    const uint32_t* wp = reinterpret_cast<const uint32_t*>(p.units) +
                         (tsvd_unit_index(tile * CLUSTER_ROWS + rp * 32, g0 + cp * GEMV_PRE, p.C_pad) + g) * 4 + q;
    uint32_t w[GEMV_PRE][2][2];
#pragma unroll
    for (int i = 0; i < GEMV_PRE; ++i) {
        const bool there = g0 + cp * GEMV_PRE + i < g1;
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int r = 0; r < 2; ++r)
                w[i][h][r] = there ? ld_stream_now(wp + i * GROUP_WORDS + (16 * h + 8 * r) * 4) : 0u;
    }
    pdl_wait();
    pdl_launch_dependents();
    tsvd_stamp_begin(p.stamp);
    PH(0);
    __syncthreads();   // the cleared maxima and counts

    // ---- this CTA's quarter of the stage input as fixed-point digits: item = (token, chunk of 8 columns) ----
    const int slab_chunks = (g1 - g0) * 8;                    // chunks of 8 columns in the slab
    const int n_items = NTOK * slab_chunks;
    constexpr int MAX_KEEP = 2;                               // items a thread keeps between the passes
    float keep[MAX_KEEP][8];
    auto load_item = [&](int it, float (&v)[8]) {
        const int b = it / slab_chunks, ch = it - b * slab_chunks;
        const IN_T* row = in + (size_t)(b < p.B ? b : 0) * p.ld_in;
        const bool vec_ok = (reinterpret_cast<uintptr_t>(row) & 15) == 0;
        load8<IN_T>(row, g0 * 64 + ch * 8, p.C, vec_ok, v);
    };
    // (all 32 lanes of a warp run the same number of trips when this holds: n_items is then a multiple of 32)
    const bool warp_one_token = (slab_chunks & 31) == 0;
    if constexpr (!kInt) {
        int k = 0;
        for (int it = tid; it < n_items; it += GEMV_THREADS, ++k) {
            float v[8];
            load_item(it, v);
            float m = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) m = fmaxf(m, fabsf(v[e]));
            if (k < MAX_KEEP) {
#pragma unroll
                for (int e = 0; e < 8; ++e) keep[k][e] = v[e];
            }
            // non-negative floats order as their bits; when a warp's 32 items belong to one token
            // (slabs of whole multiples of 256 columns) the warp reduces first
            unsigned mb = __float_as_uint(m);
            if (warp_one_token) {
                mb = __reduce_max_sync(0xffffffffu, mb);
                if (lane == 0 && mb) atomicMax(&smax[it / slab_chunks], mb);
            } else if (mb) {
                atomicMax(&smax[it / slab_chunks], mb);
            }
        }
        __syncthreads();
    }
    PH(1);
    {
        int k = 0;
        for (int it = tid; it < n_items; it += GEMV_THREADS, ++k) {
            const int b = it / slab_chunks, ch = it - b * slab_chunks;
            float v[8];
            if (!kInt && k < MAX_KEEP) {
#pragma unroll
                for (int e = 0; e < 8; ++e) v[e] = keep[k][e];
            } else {
                load_item(it, v);
            }
            uint32_t dw[ND][2];
#pragma unroll
            for (int d = 0; d < ND; ++d) dw[d][0] = dw[d][1] = 0u;
            if (b < p.B) {
                int qv[8];
                float qscale = 1.f;
                if constexpr (!kInt) {
                    const int E = tsvd_quant_exponent(__uint_as_float(smax[b]));
                    qscale = tsvd_pow2(8 * ND - 2 - E);
                    unsigned cnt = 0;
                    tsvd_range_sample(cnt, v[0], qscale);
                    if (warp_one_token) {
                        cnt = __reduce_add_sync(0xffffffffu, cnt);
                        if (lane == 0 && cnt) atomicAdd(&srange[b], cnt);
                    } else if (cnt) {
                        atomicAdd(&srange[b], cnt);
                    }
                }
                if constexpr (ND <= 3) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) qv[e] = tsvd_round_bits(v[e], qscale);
                    digits_of<ND, 2>(qv, dw, TSVD_ROUND_BIAS);
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) qv[e] = __float2int_rn(v[e] * qscale);
                    digits_of<ND, 2>(qv, dw);
                }
            }
#pragma unroll
            for (int d = 0; d < ND; ++d)
                *reinterpret_cast<uint2*>(dig + (size_t)(b * ND + d) * dstride + ch * 8) = make_uint2(dw[d][0], dw[d][1]);
        }
    }
    if (tid < NTOK) {
        float sc = 1.f;
        if constexpr (!kInt) sc = tsvd_pow2(tsvd_quant_exponent(__uint_as_float(smax[tid])) - (8 * ND - 2));
        scale[tid] = sc;
    }
    __syncthreads();
    if constexpr (!kInt) {
        if (tid < NTOK) {   // range diagnostic on this CTA's samples of the token
            const unsigned tot = srange[tid], nz = tot & 0xffffu, big = tot >> 16;
            if (nz >= 32u && 4u * big < nz) atomicOr(p.status, TSVD_DEV_RANGE);
        }
    }

    PH(2);
    // ---- stream the codes of this warp's rows and column part ----
    int acc[2][NT][4];
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[h][j][c] = 0;
    bool col_there[NT];
#pragma unroll
    for (int j = 0; j < NT; ++j) col_there[j] = 8 * j + g < NCOL;
    const int8_t* dp = dig + (size_t)g * dstride + cp * (GEMV_PRE * 64) + q * 16;
    constexpr int ROUND = 4 * GEMV_PRE;     // column groups the CTA's four column parts cover per round
#pragma unroll 1
    for (int rb = g0; rb < g1; rb += ROUND) {
        const int first = rb + cp * GEMV_PRE;          // this warp's first group of the round
        wp += ROUND * GROUP_WORDS;
        const bool more = rb + ROUND < g1;
#pragma unroll
        for (int i = 0; i < GEMV_PRE; ++i) {
            if (first + i < g1) {
                uint32_t e0[2][4], e1[2][4];   // sixteen entries of rows 16h + g and 16h + g + 8 as int8
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    tsvd_expand16(w[i][h][0], e0[h]);
                    tsvd_expand16(w[i][h][1], e1[h]);
                    if (more && first + ROUND + i < g1) {   // the group's codes are expanded: request the next round's
#pragma unroll
                        for (int r = 0; r < 2; ++r) w[i][h][r] = ld_stream_now(wp + i * GROUP_WORDS + (16 * h + 8 * r) * 4);
                    }
                }
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    // digits of columns 16q .. 16q+15 of this group, (token, digit) pair 8j + g
                    const uint4 xd = col_there[j] ? *reinterpret_cast<const uint4*>(dp + (size_t)(8 * j) * dstride + i * 64)
                                                  : make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        mma_s8(acc[h][j], e0[h][0], e1[h][0], e0[h][1], e1[h][1], xd.x, xd.y);
                        mma_s8(acc[h][j], e0[h][2], e1[h][2], e0[h][3], e1[h][3], xd.z, xd.w);
                    }
                }
            }
        }
        dp += ROUND * 64;
    }
    PH(3);
    // every warp owns its rows of its column part's plane of `red`: plain stores, summed below
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int n = 8 * j + 2 * q + (c & 1), r = rp * 32 + 16 * h + g + 8 * (c >> 1);
                if (n < NCOL) red[(cp * NCOL + n) * CLUSTER_ROWS + r] = acc[h][j][c];
            }
    __syncthreads();
    PH(4);

    // ---- this CTA's partial result of every row goes to the CTA that finishes the row ----
    for (int it = tid; it < NTOK * CLUSTER_ROWS; it += GEMV_THREADS) {
        const int b = it / CLUSTER_ROWS, r = it % CLUSTER_ROWS;
        int a[ND];
#pragma unroll
        for (int d = 0; d < ND; ++d) {   // the four column parts: exact integer additions
            const int* rr = red + (b * ND + d) * CLUSTER_ROWS + r;
            a[d] = rr[0] + rr[NCOL * CLUSTER_ROWS] + rr[2 * NCOL * CLUSTER_ROWS] + rr[3 * NCOL * CLUSTER_ROWS];
        }
        uint32_t bits;
        if constexpr (kIntSlots) {
            bits = (uint32_t)a[0];
        } else {
            float f;
            if constexpr (ND == 1) f = (float)a[0];
            else if constexpr (ND == 2) f = (float)(a[0] + (a[1] << 8));
            else {
                const int lo = a[0] + (a[1] << 8);
                int hi = a[2];
                if constexpr (ND == 4) hi += a[3] << 8;
                f = fmaf((float)hi, 65536.f, (float)lo);
            }
            bits = __float_as_uint(f * scale[b]);   // a power of two: exact
        }
        const uint32_t owner = (uint32_t)(r / CLUSTER_OWN);
        cluster_store(cluster_map(slots + ((int)rank * NTOK + b) * CLUSTER_OWN + (r % CLUSTER_OWN), owner), bits);
    }
    cluster_barrier();
    PH(5);

    // ---- thread (token, own row): the four partial results in a fixed order -> the stage's output ----
    if (tid < NTOK * CLUSTER_OWN) {
        const int b = tid / CLUSTER_OWN, r = tid % CLUSTER_OWN;
        const int orow = tile * CLUSTER_ROWS + (int)rank * CLUSTER_OWN + r;
        if (b < p.B) {
            float val;
            int zi = 0;
            if constexpr (kIntSlots) {
#pragma unroll
                for (int c = 0; c < CLUSTER_CTAS; ++c) zi += (int)slots[(c * NTOK + b) * CLUSTER_OWN + r];
                val = (float)zi;
            } else {
                val = 0.f;
#pragma unroll
                for (int c = 0; c < CLUSTER_CTAS; ++c) val += __uint_as_float(slots[(c * NTOK + b) * CLUSTER_OWN + r]);
            }
            if constexpr (STAGE == STAGE_V) {
                reinterpret_cast<float*>(p.out)[(size_t)b * p.ld_out + orow] = p.S[orow] * val;   // the K multiplications
                if (p.z_out && orow < p.R) {
                    if (p.z_int) reinterpret_cast<int*>(p.z_out)[(size_t)b * p.z_ld + orow] = zi;
                    else reinterpret_cast<float*>(p.z_out)[(size_t)b * p.z_ld + orow] = val;
                }
            } else if (orow < p.R) {
                const float yv = p.bias ? val + __ldg(p.bias + orow) : val;
                if (p.out_bf16)
                    reinterpret_cast<__nv_bfloat16*>(p.out)[(size_t)b * p.ld_out + orow] = __float2bfloat16_rn(yv);
                else
                    reinterpret_cast<float*>(p.out)[(size_t)b * p.ld_out + orow] = yv;
            }
        }
    }
    tsvd_stamp_end(p.stamp);
}

size_t gemv_cluster_smem_bytes(int nd, int ntok, int C_pad)
{
    const size_t ncol = (size_t)ntok * nd;
    return ncol * (cluster_slab_groups(C_pad) * 64 + GEMV_DIG_PAD) + 4 * ncol * CLUSTER_ROWS * sizeof(int) +
           (size_t)CLUSTER_CTAS * ntok * CLUSTER_OWN * 4 + (size_t)ntok * 12;
}
// (at one and two tokens the exchange between the four CTAs costs more than the shared conversion saves)
inline bool use_cluster_form(int C_pad, int B) { return B >= CLUSTER_MIN_TOKENS && (C_pad >> 6) >= CLUSTER_MIN_GROUPS; }

size_t gemv_smem_bytes(int nd, int ntok, int C_pad)
{
    return (size_t)ntok * nd * (C_pad + GEMV_DIG_PAD) + (size_t)ntok * nd * GEMV_ROWS * sizeof(int) +
           (size_t)ntok * sizeof(float) + (size_t)GEMV_WARPS * ntok * sizeof(float);
}

// One and two tokens take the cluster form only where the digits of a whole row do not fit one CTA's shared
// memory (contractions of tens of thousands of columns) while a quarter of them does.
inline bool stage_in_cluster_form(int nd, int C_pad, int B)
{
    if (use_cluster_form(C_pad, B)) return true;
    return B <= 2 && (C_pad >> 6) >= CLUSTER_MIN_GROUPS && gemv_smem_bytes(nd, B, C_pad) > (size_t)GEMV_MAX_SMEM;
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
    PdlLaunch cfg((unsigned)(R_pad / GEMV_ROWS), (unsigned)GEMV_THREADS, smem, stream);
    const cudaError_t e = cudaLaunchKernelEx(&cfg.cfg, ternary_gemv_kernel<IN_T, ND, NTOK, STAGE>, (const GemvParams)p);
    tsvd_count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename IN_T, int ND, int NTOK, int STAGE>
cudaError_t launch_gemv_cluster(const GemvParams& p, int R_pad, cudaStream_t stream)
{
    static bool attr_set[64] = {};   // per instantiation and device
    const size_t smem = gemv_cluster_smem_bytes(ND, NTOK, p.C_pad);
    int dev = 0;
    cudaError_t e0 = cudaGetDevice(&dev);
    if (e0 != cudaSuccess) return e0;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(ternary_gemv_cluster_kernel<IN_T, ND, NTOK, STAGE>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, GEMV_MAX_SMEM);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(R_pad / CLUSTER_ROWS * CLUSTER_CTAS));
    cfg.blockDim = dim3(GEMV_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CLUSTER_CTAS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, ternary_gemv_cluster_kernel<IN_T, ND, NTOK, STAGE>, (const GemvParams)p);
    tsvd_count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename IN_T, int ND, int STAGE>
cudaError_t launch_gemv_tokens(const GemvParams& p, int R_pad, cudaStream_t stream)
{
    if (stage_in_cluster_form(ND, p.C_pad, p.B)) {
        if (p.B == 1) return launch_gemv_cluster<IN_T, ND, 1, STAGE>(p, R_pad, stream);
        if (p.B == 2) return launch_gemv_cluster<IN_T, ND, 2, STAGE>(p, R_pad, stream);
        if (p.B <= 4) return launch_gemv_cluster<IN_T, ND, 4, STAGE>(p, R_pad, stream);
        if (p.B <= 6) return launch_gemv_cluster<IN_T, ND, 6, STAGE>(p, R_pad, stream);
        if (p.B <= 8) return launch_gemv_cluster<IN_T, ND, 8, STAGE>(p, R_pad, stream);
        if (p.B <= 12) return launch_gemv_cluster<IN_T, ND, 12, STAGE>(p, R_pad, stream);
        return launch_gemv_cluster<IN_T, ND, 16, STAGE>(p, R_pad, stream);
    }
    if (p.B > 8) return cudaErrorInvalidValue;   // (tsvd_decode_fits keeps such requests away)
    if (p.B == 1) return launch_gemv<IN_T, ND, 1, STAGE>(p, R_pad, stream);
    if (p.B == 2) return launch_gemv<IN_T, ND, 2, STAGE>(p, R_pad, stream);
    if (p.B <= 4) return launch_gemv<IN_T, ND, 4, STAGE>(p, R_pad, stream);
    return launch_gemv<IN_T, ND, 8, STAGE>(p, R_pad, stream);
}

constexpr int ND_T = 4;   // digits of the intermediate t (fp32), as on the tensor-core path
inline int digits_for_x(tsvd_dtype_t dt, bool wide) { return dt == TSVD_I8 ? 1 : (dt == TSVD_BF16 && !wide) ? 3 : 4; }

}  // namespace

bool tsvd_decode_fits(const tsvd_handle_s* h, int B, tsvd_dtype_t dt, bool wide_x)
{
    if (B < 1 || B > TSVD_DECODE_MAX_B) return false;
    int ntok = B <= 2 ? B : B <= 4 ? 4 : B <= 8 ? 8 : B <= 12 ? 12 : 16;   // tokens of the instantiation that serves B
    // nine to sixteen tokens: the cluster form only
    if (B > 8 && !(use_cluster_form(h->V.C_pad, B) && use_cluster_form(h->U.C_pad, B))) return false;
    auto need = [&](int nd, int C_pad) {
        if (!stage_in_cluster_form(nd, C_pad, B)) return gemv_smem_bytes(nd, ntok, C_pad);
        return gemv_cluster_smem_bytes(nd, (B == 5 || B == 6) ? 6 : ntok, C_pad);   // (the cluster form also has six)
    };
    return need(digits_for_x(dt, wide_x), h->V.C_pad) <= (size_t)GEMV_MAX_SMEM && need(ND_T, h->U.C_pad) <= (size_t)GEMV_MAX_SMEM;
}

bool tsvd_decode_cluster_form(const tsvd_handle_s* h, int B)
{
    return use_cluster_form(h->V.C_pad, B) && use_cluster_form(h->U.C_pad, B);
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
    p.status = h->dev_status; p.stamp = h->prof.slot(1);
    cudaError_t e;
    h->prof.begin(1, st);
    switch (a.dtype) {
        case TSVD_F32: e = launch_gemv_tokens<float, 4, STAGE_V>(p, h->V.R_pad, st); break;
        case TSVD_BF16:
            e = a.wide_x ? launch_gemv_tokens<__nv_bfloat16, 4, STAGE_V>(p, h->V.R_pad, st)
                         : launch_gemv_tokens<__nv_bfloat16, 3, STAGE_V>(p, h->V.R_pad, st);
            break;
        case TSVD_I8: e = launch_gemv_tokens<int8_t, 1, STAGE_V>(p, h->V.R_pad, st); break;
        default: return TSVD_E_DTYPE;
    }
    h->prof.end(st);
    if (e != cudaSuccess) return TSVD_E_CUDA;
    if (a.v_only) { *a.t_where = t; return TSVD_OK; }

    GemvParams q{};
    q.units = h->U.units; q.R = h->M; q.C = h->K; q.C_pad = h->U.C_pad;
    q.in = t; q.ld_in = h->V.R_pad; q.B = a.B;
    q.out = a.y; q.ld_out = a.ldy;
    q.out_bf16 = (a.dtype == TSVD_BF16) && !a.out_f32;
    q.bias = h->bias; q.status = h->dev_status; q.stamp = h->prof.slot(3);
    h->prof.begin(3, st);
    e = launch_gemv_tokens<float, ND_T, STAGE_U>(q, h->U.R_pad, st);
    h->prof.end(st);
    return e == cudaSuccess ? TSVD_OK : TSVD_E_CUDA;
}
