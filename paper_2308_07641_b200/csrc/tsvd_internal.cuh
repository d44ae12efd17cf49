// Internal definitions shared by the libtsvd translation units (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <type_traits>
#include <vector>

#include "tsvd.h"

// ---------------------------------------------------------------------------------------
// Packed ternary format (2 bits per entry: bit0 = nonzero, bit1 = sign, code 2 never used;
// +1 -> 1, -1 -> 3, 0 -> 0).  The paper fixes only "2 bits per element"; the arrangement
// below is chosen for the kernels.
//
// A ternary matrix T [R, C] (R = output rows, C = contraction index; this is V [K,N]
// and U [M,K] as they are) is padded to R_pad (multiple of 128) x C_pad (multiple of
// 128) and cut into blocks of 128 rows x 64 columns.  Block (rt, cg) occupies 2 KiB at
// unit index (rt * (C_pad/64) + cg) * 128; inside it row r (0..127) owns one 16-byte
// unit = 4 words; word w covers columns cg*64 + 16*w .. +15.  Inside a word, entry e
// (0..15) sits at bits [4e, 4e+1] for e < 8 and at bits [4(e-8)+2, 4(e-8)+3] for e >= 8,
// so that (w & 0x33333333) and ((w >> 2) & 0x33333333) are directly byte-permute
// selectors that expand eight entries each into int8 lanes.
//
// Consequences: a 128-row x 128-column MMA operand tile is 4 KiB contiguous; consecutive
// rows of one 64-column group are consecutive 16-byte units (coalesced 128-bit loads when
// a thread owns a row).
// ---------------------------------------------------------------------------------------
constexpr int TSVD_ROW_TILE = 128;
constexpr int TSVD_COL_GROUP = 64;
constexpr int TSVD_COL_PAD = 128;

struct PackedMat {
    uint4* units = nullptr;  // device
    int R = 0, C = 0;        // logical
    int R_pad = 0, C_pad = 0;
    size_t n_units = 0;      // R_pad * C_pad / 64
    unsigned long long nnz = 0;
    size_t bytes() const { return n_units * sizeof(uint4); }
};

// Index-list form of a ternary matrix (index.cu): per row the list of its nonzeros.
struct IndexMat {
    int* row_ptr = nullptr;        // device, [R + 1]
    uint16_t* entries = nullptr;   // device, [nnz]: (column << 1) | (1 if the entry is -1)
    int R = 0, C = 0, C_pad = 0;
    size_t nnz = 0;
    size_t bytes() const { return row_ptr ? ((size_t)R + 1) * sizeof(int) + nnz * sizeof(uint16_t) : 0; }
};

__host__ __device__ inline size_t tsvd_unit_index(int row, int col_group, int C_pad)
{
    return ((size_t)(row >> 7) * (size_t)(C_pad >> 6) + (size_t)col_group) * 128 + (size_t)(row & 127);
}

// bit position of entry e (0..15) inside its word
__host__ __device__ inline int tsvd_entry_shift(int e) { return (e < 8) ? 4 * e : 4 * (e - 8) + 2; }

// Expand eight 2-bit codes (selector nibbles, see above) to eight int8 values:
// lo word = entries 0..3, hi word = entries 4..7 of the selector.
__device__ __forceinline__ void tsvd_expand8(uint32_t sel, uint32_t& lo, uint32_t& hi)
{
    // byte table: code 0 -> 0x00, 1 -> 0x01, 2 -> 0x00, 3 -> 0xFF
    const uint32_t table = 0xFF000100u;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(lo) : "r"(table), "r"(0u), "r"(sel));
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(table), "r"(0u), "r"(sel >> 16));
}

// Expand one packed word to sixteen int8 values (four 32-bit lanes, entries in order).
__device__ __forceinline__ void tsvd_expand16(uint32_t w, uint32_t out[4])
{
    tsvd_expand8(w & 0x33333333u, out[0], out[1]);
    tsvd_expand8((w >> 2) & 0x33333333u, out[2], out[3]);
}

// Per-kernel timing behind tsvd_profile_enable / tsvd_profile_read.  Mode 1: a CUDA-event pair
// around every launch (eager streams only; a pair carries the launch latency).  Mode 2: the kernels
// themselves write the global nanosecond timer into a pair of words per launch -- the first CTA when
// its wait for the previous kernel ends, every warp when it finishes (maximum) -- which also works
// inside a captured graph: each captured launch keeps its own pair and every replay overwrites it
// (the timer only grows, so the maximum needs no reset).
struct StageProfiler {
    int mode = 0;
    bool on = false;            // mode 1
    struct Pair { cudaEvent_t a, b; int stage; };
    std::vector<Pair> pending;
    float ms[TSVD_N_STAGES] = {0, 0, 0, 0};
    unsigned launches[TSVD_N_STAGES] = {0, 0, 0, 0};
    unsigned long long* stamps = nullptr;   // mode 2: device, [TSVD_STAMP_SLOTS][TSVD_STAMP_WORDS]: begin, end, spare
    std::vector<int> slot_stage;            // stage of every slot handed out
    void begin(int stage, cudaStream_t s);
    void end(cudaStream_t s);
    void drain();
    unsigned long long* slot(int stage);    // mode 2: this launch's pair (null when off or full)
};
constexpr int TSVD_STAMP_SLOTS = 1 << 15;
constexpr int TSVD_STAMP_WORDS = 8;   // begin, end, and six spare words for finer stamps in development builds

struct tsvd_handle_s {
    int device = 0;
    int M = 0, K = 0, N = 0;
    PackedMat V;          // rows K, contraction N
    PackedMat U;          // rows M, contraction K
    float* S = nullptr;   // device, length V.R_pad (zero padded)
    float* bias = nullptr;  // device, length U.R_pad (zero padded), or null: no bias
    IndexMat Vi, Ui;      // only with TSVD_PACK_INDEX_LISTS
    // scratch shared by all forwards on this handle
    void* ws = nullptr;
    size_t ws_bytes = 0;
    void* io = nullptr;   // device staging for the host-buffer entry point
    size_t io_bytes = 0;
    cudaStream_t host_stream[3] = {nullptr, nullptr, nullptr};   // copy-in, compute, copy-out of the host-buffer entry point
    std::vector<cudaEvent_t> host_events;
    int* dev_status = nullptr;  // device status word: TSVD_DEV_* bits
    StageProfiler prof;
};

// bits of the device status word
constexpr int TSVD_DEV_TIMEOUT = 1;   // a bounded wait gave up
constexpr int TSVD_DEV_RANGE = 2;     // a token's dynamic range exceeded what the digits resolve
constexpr int TSVD_DEV_BOUNDS = 4;    // checked builds (-DTSVD_CHECK_BOUNDS): a ring or tile index left its range

// Index checks of the contraction kernel's rings and tiles, compiled in with -DTSVD_CHECK_BOUNDS: a
// violated bound raises TSVD_DEV_BOUNDS in the device status word (and nothing else: the access still
// happens, so a checked build is for finding a wrong index, not for surviving one).
#ifdef TSVD_CHECK_BOUNDS
#define TSVD_BOUND(status, cond) do { if (!(cond)) atomicOr((status), TSVD_DEV_BOUNDS); } while (0)
#else
#define TSVD_BOUND(status, cond) do { } while (0)
#endif

// Programmatic dependent launch: a kernel launched with this configuration may be set up, and
// run up to its pdl_wait(), while the kernel before it in the stream is still running;
// pdl_wait() returns once that kernel has completed and its writes are visible.  A kernel calls
// pdl_launch_dependents() to let the kernel after it start likewise.  Without the launch
// attribute (or with nothing before or after it) both calls do nothing.
struct PdlLaunch {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    PdlLaunch(unsigned grid, unsigned block, size_t smem, cudaStream_t stream)
    {
        cfg = cudaLaunchConfig_t{};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(block);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    PdlLaunch(const PdlLaunch&) = delete;
    PdlLaunch& operator=(const PdlLaunch&) = delete;
};
#ifdef __CUDACC__
__device__ __forceinline__ unsigned long long tsvd_globaltimer()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Time stamps of one launch (see StageProfiler, mode 2); `s` is null unless profiling is on.
__device__ __forceinline__ void tsvd_stamp_begin(unsigned long long* s)
{
    if (s && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) s[0] = tsvd_globaltimer();
}
// the same from any one warp of the grid's first CTA (lane 0 writes)
__device__ __forceinline__ void tsvd_stamp_begin_any(unsigned long long* s)
{
    if (s && blockIdx.x == 0 && blockIdx.y == 0 && (threadIdx.x & 31) == 0) s[0] = tsvd_globaltimer();
}
__device__ __forceinline__ void tsvd_stamp_end(unsigned long long* s)   // every warp, at its end
{
    if (s && (threadIdx.x & 31) == 0) atomicMax(s + 1, tsvd_globaltimer());
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif

// launch accounting
void tsvd_count_launch(unsigned n = 1);

// pack.cu
tsvd_status_t tsvd_pack_matrix(const int8_t* host, int R, int C, PackedMat* out, int* dev_flag);
tsvd_status_t tsvd_unpack_matrix(const PackedMat& pm, int8_t* host);

// simple.cu -- CUDA-core reference kernels
// A stage input given as the patches of an NHWC image batch instead of a matrix: token b = (n, ho, wo)
// reads, for kernel position (a, b2), the C channels of pixel (ho*sh + a*dh - ph, wo*sw + b2*dw - pw) of
// image n (zeros outside the image); its row is the k1*k2 runs of C values in the order (a, b2, channel).
// C = 0: off.  C is a multiple of 16, so that a 16-value chunk never straddles two runs.
struct PatchGather {
    int H = 0, W = 0, C = 0, k2 = 0, sh = 0, sw = 0, ph = 0, pw = 0, dh = 0, dw = 0, Ho = 0, Wo = 0, feat = 0;
};
#ifdef __CUDACC__
// Where the values feat0 .. (a chunk inside one run) of token (n, ho, wo) lie; null outside the image.
template <typename T>
__device__ __forceinline__ const T* tsvd_patch_ptr(const PatchGather& g, const T* img, int n, int ho, int wo, int feat0)
{
    const int ab = feat0 / g.C, c0 = feat0 - ab * g.C;
    const int a = ab / g.k2, b2 = ab - a * g.k2;
    const int h = ho * g.sh + a * g.dh - g.ph, w = wo * g.sw + b2 * g.dw - g.pw;
    if (h < 0 || h >= g.H || w < 0 || w >= g.W) return nullptr;
    return img + (((long long)n * g.H + h) * g.W + w) * g.C + c0;
}
#endif

struct ForwardArgs {
    tsvd_handle_s* h;
    const void* x;
    int ldx;
    void* y;
    int ldy;
    int B;
    tsvd_dtype_t dtype;
    bool out_f32;
    void* z_out;
    bool test_stall = false;   // TSVD_FLAG_TEST_STALL
    bool wide_x = false;       // TSVD_FLAG_WIDE_X: bf16 activations as four digits
    bool v_only = false;       // stop after the V-stage and its scale (tsvd_forward_v)
    float** t_where = nullptr; // v_only: receives where t = S*(V x) was written, [B][R_pad of V] fp32
    const PatchGather* gather = nullptr;   // the tokens are patches of the image batch at x (tensor-core path only)
    float* t;        // scratch [B][t_ld] fp32: S * (V x)
    int t_ld;
    cudaStream_t stream;
};
tsvd_status_t tsvd_forward_simple(const ForwardArgs& a);
size_t tsvd_simple_ws_bytes(const tsvd_handle_s* h, int B);

// tensor.cu -- tcgen05 path
tsvd_status_t tsvd_forward_tensor(const ForwardArgs& a, void* ws);
size_t tsvd_tensor_ws_bytes(const tsvd_handle_s* h, int B, tsvd_dtype_t dt, bool wide_x);
size_t tsvd_tensor_ws_bytes_upto(const tsvd_handle_s* h, int B_max, tsvd_dtype_t dt, bool wide_x);
int tsvd_tensor_digits_x(tsvd_dtype_t dt, bool wide_x);
int tsvd_tensor_digits_t();

// midbatch.cu -- five to thirty-two tokens: one launch per stage, clusters share a row tile's contraction
bool tsvd_mid_fits(const tsvd_handle_s* h, int B, tsvd_dtype_t dt, bool wide_x);
size_t tsvd_mid_ws_bytes(const tsvd_handle_s* h, int B);
tsvd_status_t tsvd_forward_mid(const ForwardArgs& a, void* ws);

// decode.cu -- one to sixteen tokens, bound by streaming the packed codes
bool tsvd_decode_fits(const tsvd_handle_s* h, int B, tsvd_dtype_t dt, bool wide_x);
bool tsvd_decode_cluster_form(const tsvd_handle_s* h, int B);   // both stages would run the cluster form
size_t tsvd_decode_ws_bytes(const tsvd_handle_s* h, int B);
tsvd_status_t tsvd_forward_decode(const ForwardArgs& a, void* ws);

// index.cu -- index-list form for very sparse rows, one to four tokens
tsvd_status_t tsvd_build_index_lists(const int8_t* host, int R, int C, IndexMat* out);
bool tsvd_index_fits(const tsvd_handle_s* h, int B);
tsvd_status_t tsvd_forward_index(const ForwardArgs& a, void* ws);

#define TSVD_CUDA_OK(expr)                            \
    do {                                              \
        cudaError_t _e = (expr);                      \
        if (_e != cudaSuccess) {                      \
            (void)cudaGetLastError();                 \
            return (_e == cudaErrorMemoryAllocation) ? TSVD_E_NOMEM : TSVD_E_CUDA; \
        }                                             \
    } while (0)
