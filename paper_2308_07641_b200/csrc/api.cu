// The C ABI of libtsvd (see include/tsvd.h): argument validation, handle lifetime,
// scratch management and dispatch.  No arithmetic of the map is done on the host.
#include <atomic>
#include <new>

#include "tsvd_internal.cuh"

static std::atomic<unsigned long long> g_launches{0};
void tsvd_count_launch(unsigned n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

extern "C" unsigned long long tsvd_launch_count(void) { return g_launches.load(); }

extern "C" const char* tsvd_strerror(tsvd_status_t s)
{
    switch (s) {
        case TSVD_OK: return "ok";
        case TSVD_E_NULL: return "null pointer argument";
        case TSVD_E_SHAPE: return "bad shape, batch or leading dimension";
        case TSVD_E_VALUE: return "U or V holds a value outside {-1,0,+1}";
        case TSVD_E_DTYPE: return "unknown dtype or unsupported flags";
        case TSVD_E_ALIGN: return "pointer or leading dimension not aligned as required";
        case TSVD_E_CUDA: return "CUDA runtime error (or no CUDA device)";
        case TSVD_E_TIMEOUT: return "a bounded device-side wait gave up";
        case TSVD_E_NOMEM: return "out of memory";
        case TSVD_E_TOOBIG: return "request exceeds a fixed capacity (static scratch, contraction length or index width)";
        case TSVD_E_RANGE: return "a token's dynamic range exceeded what the fixed-point digits resolve";
        case TSVD_E_INTERNAL: return "a checked build found an index outside its range";
    }
    return "unknown status";
}

void StageProfiler::begin(int stage, cudaStream_t s)
{
    if (!on) return;
    if (pending.size() >= 8192) drain();
    Pair p;
    p.stage = stage;
    if (cudaEventCreate(&p.a) != cudaSuccess || cudaEventCreate(&p.b) != cudaSuccess) { (void)cudaGetLastError(); return; }
    cudaEventRecord(p.a, s);
    pending.push_back(p);
}

void StageProfiler::end(cudaStream_t s)
{
    if (!on || pending.empty()) return;
    cudaEventRecord(pending.back().b, s);
}

unsigned long long* StageProfiler::slot(int stage)
{
    if (mode != 2 || !stamps || slot_stage.size() >= (size_t)TSVD_STAMP_SLOTS) return nullptr;
    slot_stage.push_back(stage);
    return stamps + TSVD_STAMP_WORDS * (slot_stage.size() - 1);
}

void StageProfiler::drain()
{
    for (auto& p : pending) {
        float t = 0.f;
        if (cudaEventSynchronize(p.b) == cudaSuccess && cudaEventElapsedTime(&t, p.a, p.b) == cudaSuccess) {
            ms[p.stage] += t;
            launches[p.stage] += 1;
        }
        cudaEventDestroy(p.a);
        cudaEventDestroy(p.b);
    }
    (void)cudaGetLastError();
    pending.clear();
}

extern "C" tsvd_status_t tsvd_profile_enable(tsvd_handle_t h, int mode)
{
    if (!h) return TSVD_E_NULL;
    if (mode < 0 || mode > 2) return TSVD_E_DTYPE;
    h->prof.drain();
    for (int i = 0; i < TSVD_N_STAGES; ++i) { h->prof.ms[i] = 0.f; h->prof.launches[i] = 0; }
    h->prof.slot_stage.clear();
    h->prof.mode = mode;
    h->prof.on = mode == 1;
    if (mode == 2) {
        const size_t bytes = (size_t)TSVD_STAMP_SLOTS * TSVD_STAMP_WORDS * sizeof(unsigned long long);
        if (!h->prof.stamps && cudaMalloc(&h->prof.stamps, bytes) != cudaSuccess) {
            (void)cudaGetLastError();
            h->prof.stamps = nullptr;
            h->prof.mode = 0;
            return TSVD_E_NOMEM;
        }
        TSVD_CUDA_OK(cudaMemset(h->prof.stamps, 0, bytes));
    }
    return TSVD_OK;
}

#ifdef TSVD_PHASES
// development builds only: the raw words of the first `n` recorded launches and their stages
extern "C" int tsvd_debug_phases(tsvd_handle_t h, unsigned long long* out, int* stages, int n)
{
    cudaDeviceSynchronize();
    const int have = (int)h->prof.slot_stage.size();
    if (n > have) n = have;
    cudaMemcpy(out, h->prof.stamps, (size_t)n * TSVD_STAMP_WORDS * sizeof(unsigned long long), cudaMemcpyDeviceToHost);
    for (int i = 0; i < n; ++i) stages[i] = h->prof.slot_stage[i];
    return n;
}
#endif

extern "C" tsvd_status_t tsvd_profile_read(tsvd_handle_t h, float* ms_sum, unsigned* launches)
{
    if (!h || !ms_sum || !launches) return TSVD_E_NULL;
    if (h->prof.mode == 2) {
        // the pairs of every launch recorded since tsvd_profile_enable, as the kernels last wrote them
        const size_t n = h->prof.slot_stage.size();
        std::vector<unsigned long long> host(TSVD_STAMP_WORDS * n + 2);
        TSVD_CUDA_OK(cudaDeviceSynchronize());
        if (n) TSVD_CUDA_OK(cudaMemcpy(host.data(), h->prof.stamps, TSVD_STAMP_WORDS * n * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
        for (int i = 0; i < TSVD_N_STAGES; ++i) { ms_sum[i] = 0.f; launches[i] = 0; }
        double ns[TSVD_N_STAGES] = {0, 0, 0, 0};
        for (size_t i = 0; i < n; ++i) {
            const unsigned long long b = host[TSVD_STAMP_WORDS * i], e = host[TSVD_STAMP_WORDS * i + 1];
            if (b == 0 || e <= b) continue;     // never ran
            ns[h->prof.slot_stage[i]] += (double)(e - b);
            launches[h->prof.slot_stage[i]] += 1;
        }
        for (int i = 0; i < TSVD_N_STAGES; ++i) ms_sum[i] = (float)(ns[i] * 1e-6);
        return TSVD_OK;
    }
    h->prof.drain();
    for (int i = 0; i < TSVD_N_STAGES; ++i) {
        ms_sum[i] = h->prof.ms[i];
        launches[i] = h->prof.launches[i];
        h->prof.ms[i] = 0.f;
        h->prof.launches[i] = 0;
    }
    return TSVD_OK;
}

static void free_handle(tsvd_handle_s* h)
{
    if (!h) return;
    h->prof.drain();
    if (h->V.units) cudaFree(h->V.units);
    if (h->U.units) cudaFree(h->U.units);
    if (h->S) cudaFree(h->S);
    if (h->bias) cudaFree(h->bias);
    for (IndexMat* im : {&h->Vi, &h->Ui}) {
        if (im->row_ptr) cudaFree(im->row_ptr);
        if (im->entries) cudaFree(im->entries);
    }
    if (h->ws) cudaFree(h->ws);
    if (h->io) cudaFree(h->io);
    if (h->dev_status) cudaFree(h->dev_status);
    if (h->prof.stamps) cudaFree(h->prof.stamps);
    for (cudaEvent_t e : h->host_events) cudaEventDestroy(e);
    for (cudaStream_t st : h->host_stream)
        if (st) cudaStreamDestroy(st);
    (void)cudaGetLastError();
    delete h;
}

extern "C" void tsvd_destroy(tsvd_handle_t h)
{
    if (!h) return;
    const int dev = h->device;
    int prev = dev;
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) cudaSetDevice(dev);
    cudaDeviceSynchronize();
    free_handle(h);
    if (prev != dev) cudaSetDevice(prev);
}

extern "C" tsvd_status_t tsvd_pack(const int8_t* U, const float* S, const int8_t* V, int M, int K, int N,
                                   unsigned flags, tsvd_handle_t* out)
{
    if (!out) return TSVD_E_NULL;
    *out = nullptr;
    if (!U || !S || !V) return TSVD_E_NULL;
    if (M < 1 || K < 1 || N < 1) return TSVD_E_SHAPE;
    if (flags & ~TSVD_PACK_INDEX_LISTS) return TSVD_E_DTYPE;
    // the digit sums of a row are combined in 32-bit integers: bound the contraction length
    if (N > TSVD_MAX_CONTRACTION || K > TSVD_MAX_CONTRACTION) return TSVD_E_TOOBIG;
    if ((flags & TSVD_PACK_INDEX_LISTS) && (N > TSVD_INDEX_MAX_COLUMNS || K > TSVD_INDEX_MAX_COLUMNS)) return TSVD_E_TOOBIG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return TSVD_E_CUDA; }

    tsvd_handle_s* h = new (std::nothrow) tsvd_handle_s();
    if (!h) return TSVD_E_NOMEM;
    h->device = dev;
    h->M = M; h->K = K; h->N = N;

    tsvd_status_t st = TSVD_OK;
    do {
        if (cudaMalloc(&h->dev_status, sizeof(int)) != cudaSuccess) { st = TSVD_E_NOMEM; break; }
        if (cudaMemset(h->dev_status, 0, sizeof(int)) != cudaSuccess) { st = TSVD_E_CUDA; break; }
        if ((st = tsvd_pack_matrix(V, K, N, &h->V, h->dev_status)) != TSVD_OK) break;
        if ((st = tsvd_pack_matrix(U, M, K, &h->U, h->dev_status)) != TSVD_OK) break;
        int flag = 0;
        if (cudaMemcpy(&flag, h->dev_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) {
            st = TSVD_E_CUDA; break;
        }
        if (flag) { st = TSVD_E_VALUE; break; }
        if (flags & TSVD_PACK_INDEX_LISTS) {
            if ((st = tsvd_build_index_lists(V, K, N, &h->Vi)) != TSVD_OK) break;
            if ((st = tsvd_build_index_lists(U, M, K, &h->Ui)) != TSVD_OK) break;
        }
        const size_t s_len = (size_t)h->V.R_pad;
        if (cudaMalloc(&h->S, s_len * sizeof(float)) != cudaSuccess) { st = TSVD_E_NOMEM; break; }
        if (cudaMemset(h->S, 0, s_len * sizeof(float)) != cudaSuccess) { st = TSVD_E_CUDA; break; }
        if (cudaMemcpy(h->S, S, (size_t)K * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) {
            st = TSVD_E_CUDA; break;
        }
        if (cudaMemset(h->dev_status, 0, sizeof(int)) != cudaSuccess) { st = TSVD_E_CUDA; break; }
    } while (0);
    if (st != TSVD_OK) {
        (void)cudaGetLastError();
        free_handle(h);
        return st;
    }
    *out = h;
    return TSVD_OK;
}

extern "C" tsvd_status_t tsvd_info(tsvd_handle_t h, int* M, int* K, int* N, size_t* packed_bytes,
                                   double* density_u, double* density_v)
{
    if (!h) return TSVD_E_NULL;
    if (M) *M = h->M;
    if (K) *K = h->K;
    if (N) *N = h->N;
    if (packed_bytes) *packed_bytes = h->U.bytes() + h->V.bytes() + (size_t)h->K * sizeof(float);
    if (density_u) *density_u = (double)h->U.nnz / ((double)h->M * (double)h->K);
    if (density_v) *density_v = (double)h->V.nnz / ((double)h->K * (double)h->N);
    return TSVD_OK;
}

extern "C" tsvd_status_t tsvd_index_bytes(tsvd_handle_t h, size_t* v_bytes, size_t* u_bytes)
{
    if (!h) return TSVD_E_NULL;
    if (v_bytes) *v_bytes = h->Vi.bytes();
    if (u_bytes) *u_bytes = h->Ui.bytes();
    return TSVD_OK;
}

extern "C" tsvd_status_t tsvd_unpack(tsvd_handle_t h, int8_t* U, float* S, int8_t* V)
{
    if (!h) return TSVD_E_NULL;
    tsvd_status_t st;
    if (U && (st = tsvd_unpack_matrix(h->U, U)) != TSVD_OK) return st;
    if (V && (st = tsvd_unpack_matrix(h->V, V)) != TSVD_OK) return st;
    if (S) TSVD_CUDA_OK(cudaMemcpy(S, h->S, (size_t)h->K * sizeof(float), cudaMemcpyDeviceToHost));
    return TSVD_OK;
}

extern "C" tsvd_status_t tsvd_last_status(tsvd_handle_t h)
{
    if (!h) return TSVD_E_NULL;
    int word = 0;
    TSVD_CUDA_OK(cudaMemcpy(&word, h->dev_status, sizeof(int), cudaMemcpyDeviceToHost));
    if (word) TSVD_CUDA_OK(cudaMemset(h->dev_status, 0, sizeof(int)));
    if (word & TSVD_DEV_BOUNDS) return TSVD_E_INTERNAL;
    if (word & TSVD_DEV_TIMEOUT) return TSVD_E_TIMEOUT;
    return (word & TSVD_DEV_RANGE) ? TSVD_E_RANGE : TSVD_OK;
}

extern "C" tsvd_status_t tsvd_set_bias(tsvd_handle_t h, const float* bias)
{
    if (!h) return TSVD_E_NULL;
    TSVD_CUDA_OK(cudaDeviceSynchronize());
    if (!bias) {
        if (h->bias) { cudaFree(h->bias); h->bias = nullptr; }
        return TSVD_OK;
    }
    const size_t len = (size_t)h->U.R_pad;
    if (!h->bias && cudaMalloc(&h->bias, len * sizeof(float)) != cudaSuccess) {
        (void)cudaGetLastError();
        h->bias = nullptr;
        return TSVD_E_NOMEM;
    }
    TSVD_CUDA_OK(cudaMemset(h->bias, 0, len * sizeof(float)));
    TSVD_CUDA_OK(cudaMemcpy(h->bias, bias, (size_t)h->M * sizeof(float), cudaMemcpyHostToDevice));
    return TSVD_OK;
}

static size_t dtype_size(tsvd_dtype_t d)
{
    switch (d) {
        case TSVD_F32: return 4;
        case TSVD_BF16: return 2;
        case TSVD_I8: return 1;
    }
    return 0;
}

// Grow the handle's scratch to at least `bytes` (synchronises the device when it grows).
static tsvd_status_t ensure_ws(tsvd_handle_s* h, size_t bytes)
{
    if (bytes <= h->ws_bytes) return TSVD_OK;
    TSVD_CUDA_OK(cudaDeviceSynchronize());
    if (h->ws) { cudaFree(h->ws); h->ws = nullptr; h->ws_bytes = 0; }
    const size_t rounded = (bytes + 255) & ~(size_t)255;
    if (cudaMalloc(&h->ws, rounded) != cudaSuccess) { (void)cudaGetLastError(); return TSVD_E_NOMEM; }
    h->ws_bytes = rounded;
    return TSVD_OK;
}

// The dispatch rule shared by tsvd_plan and tsvd_forward_ex.  Up to TSVD_DECODE_MAX_B tokens run
// the decode kernels when the digits of the stage inputs fit in shared memory; everything else
// runs the tensor-core kernels (which serve every batch size); the CUDA-core kernels remain as
// the plain reference path, and the index-list kernels (handles packed with index lists, up to
// TSVD_INDEX_MAX_B tokens) are run on request.  Returns 0 when a forced path cannot serve the request.
static unsigned choose_path(const tsvd_handle_s* h, int B, tsvd_dtype_t dtype, unsigned forced, bool wide_x)
{
    if (forced == TSVD_FLAG_PATH_SIMPLE) return TSVD_FLAG_PATH_SIMPLE;
    if (forced == TSVD_FLAG_PATH_TENSOR) return TSVD_FLAG_PATH_TENSOR;
    if (forced == TSVD_FLAG_PATH_INDEX) return tsvd_index_fits(h, B) ? TSVD_FLAG_PATH_INDEX : 0u;
    const bool fits = tsvd_decode_fits(h, B, dtype, wide_x);
    if (forced == TSVD_FLAG_PATH_DECODE) return fits ? TSVD_FLAG_PATH_DECODE : 0u;
    // The cluster kernels of the tensor-core path (one launch per stage, up to thirty-two tokens) are
    // the faster ones from nine tokens on, and from five where the decode kernels would run their
    // single-CTA form (a contraction under 1024 columns): measured, bf16, microseconds per forward,
    // decode / cluster-tensor: 768^3 at 5 and 8 tokens 10.9 / 7.7 and 11.2 / 7.7; 4096^3 at 6, 8, 9 and 16
    // tokens 11.5 / 13.1, 12.9 / 13.1, 16.5 / 14.1 and 21.2 / 14.6; at four tokens and fewer the decode
    // kernels win everywhere (4096^3: 9.1 / 13.0).
    if (tsvd_mid_fits(h, B, dtype, wide_x) && (B >= 9 || !tsvd_decode_cluster_form(h, B))) return TSVD_FLAG_PATH_TENSOR;
    // Three tokens and more on tall matrices: the decode kernels run one CTA per 32 rows and SM, so a stage of
    // R rows takes ceil(R / 32 / SMs) rounds of about 3.8 us (three and four tokens), 5 us (up to eight) or 7 us
    // (up to sixteen), while one padded token tile on the tile kernels costs about 16 us plus 0.2 us per block of
    // 128 columns a CTA walks through.  Measured, decode / tiles: 32768 x 1024 x 1024 at 3 and 8 tokens 29 / 17
    // and 38 / 17 us; 16384 x 4096 x 4096 at 4, 8 and 9-16 tokens 23 / 30, 33 / 30 and 33-35 / 30; 8192^3 at
    // 4 and 9-16 tokens 29 / 43 and 41-51 / 43; 4096 x 4096 x 8192 at 9-16 tokens 23-29 / 36.
    if (fits && B >= 3) {
        int sms = 148, dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const int rv = h->V.R_pad / 128, ru = h->U.R_pad / 128;
        const int rounds = (4 * rv + sms - 1) / sms + (4 * ru + sms - 1) / sms;
        const double decode_us = rounds * (B <= 4 ? 3.8 : B <= 8 ? 5.0 : 7.0);
        const double tiles_us = 16.0 + 0.195 * ((double)((rv + sms - 1) / sms) * (h->V.C_pad / 128) +
                                                (double)((ru + sms - 1) / sms) * (h->U.C_pad / 128));
        if (decode_us > tiles_us || (B >= 9 && rounds >= 4)) return TSVD_FLAG_PATH_TENSOR;
    }
    return fits ? TSVD_FLAG_PATH_DECODE : TSVD_FLAG_PATH_TENSOR;
}

extern "C" tsvd_status_t tsvd_plan(tsvd_handle_t h, int B, tsvd_dtype_t dtype, unsigned flags, unsigned* path,
                                   int* digits_x, int* digits_t)
{
    if (!h) return TSVD_E_NULL;
    if (B < 1) return TSVD_E_SHAPE;
    if (dtype_size(dtype) == 0) return TSVD_E_DTYPE;
    const unsigned forced = flags & TSVD_FLAG_PATH_MASK;
    if (forced & (forced - 1)) return TSVD_E_DTYPE;
    const bool wide_x = (flags & TSVD_FLAG_WIDE_X) != 0;
    const unsigned p = choose_path(h, B, dtype, forced, wide_x);
    if (p == 0u) return TSVD_E_TOOBIG;
    if (path) *path = p;
    // the index-list kernels quantise by the same rule (as many bytes, not split into digits)
    if (digits_x) *digits_x = (p != TSVD_FLAG_PATH_SIMPLE) ? tsvd_tensor_digits_x(dtype, wide_x) : 0;
    if (digits_t) *digits_t = (p != TSVD_FLAG_PATH_SIMPLE) ? tsvd_tensor_digits_t() : 0;
    return TSVD_OK;
}

static tsvd_status_t forward_impl(tsvd_handle_t h, const void* x, int ldx, void* y, int ldy, int B, tsvd_dtype_t dtype,
                                  unsigned flags, void* z_out, void* stream, bool v_only, float** t_where,
                                  const PatchGather* gather = nullptr)
{
    if (!h || !x || !y) return TSVD_E_NULL;
    if (B < 1) return TSVD_E_SHAPE;
    const size_t xs = dtype_size(dtype);
    if (xs == 0) return TSVD_E_DTYPE;
    const unsigned known = TSVD_FLAG_OUT_F32 | TSVD_FLAG_PATH_MASK | TSVD_FLAG_TEST_STALL | TSVD_FLAG_WIDE_X;
    if (flags & ~known) return TSVD_E_DTYPE;
    const unsigned path = flags & TSVD_FLAG_PATH_MASK;
    if (path & (path - 1)) return TSVD_E_DTYPE;  // at most one forced path
    if (ldx < h->N || ldy < (v_only ? h->K : h->M)) return TSVD_E_SHAPE;
    if (((uintptr_t)x & 15) || ((uintptr_t)y & 15) || ((uintptr_t)z_out & 3)) return TSVD_E_ALIGN;

    int dev = 0;
    TSVD_CUDA_OK(cudaGetDevice(&dev));
    if (dev != h->device) return TSVD_E_CUDA;

    ForwardArgs a;
    a.h = h; a.x = x; a.ldx = ldx; a.y = y; a.ldy = ldy; a.B = B; a.dtype = dtype;
    a.out_f32 = (flags & TSVD_FLAG_OUT_F32) != 0;
    a.z_out = z_out;
    a.test_stall = (flags & TSVD_FLAG_TEST_STALL) != 0;
    a.wide_x = (flags & TSVD_FLAG_WIDE_X) != 0;
    a.v_only = v_only;
    a.t_where = t_where;
    a.gather = gather;
    if (v_only && path == TSVD_FLAG_PATH_INDEX) return TSVD_E_DTYPE;   // the index-list kernels run whole forwards only
    a.stream = (cudaStream_t)stream;

    const unsigned chosen = choose_path(h, B, dtype, path, a.wide_x);
    if (chosen == 0u) return TSVD_E_TOOBIG;
    if (gather && chosen != TSVD_FLAG_PATH_TENSOR) return TSVD_E_SHAPE;   // only those kernels read patches in place
    if (chosen == TSVD_FLAG_PATH_TENSOR) {
        tsvd_status_t st = ensure_ws(h, tsvd_tensor_ws_bytes(h, B, dtype, a.wide_x));
        if (st != TSVD_OK) return st;
        return tsvd_forward_tensor(a, h->ws);
    }
    if (chosen == TSVD_FLAG_PATH_DECODE) {
        tsvd_status_t st = ensure_ws(h, tsvd_decode_ws_bytes(h, B));
        if (st != TSVD_OK) return st;
        return tsvd_forward_decode(a, h->ws);
    }
    if (chosen == TSVD_FLAG_PATH_INDEX) {
        tsvd_status_t st = ensure_ws(h, tsvd_decode_ws_bytes(h, B));   // the same t [B][K padded]
        if (st != TSVD_OK) return st;
        return tsvd_forward_index(a, h->ws);
    }
    tsvd_status_t st = ensure_ws(h, tsvd_simple_ws_bytes(h, B));
    if (st != TSVD_OK) return st;
    a.t = reinterpret_cast<float*>(h->ws);
    a.t_ld = h->V.R_pad;
    return tsvd_forward_simple(a);
}

extern "C" tsvd_status_t tsvd_forward_ex(tsvd_handle_t h, const void* x, int ldx, void* y, int ldy, int B,
                                         tsvd_dtype_t dtype, unsigned flags, void* z_out, void* stream)
{
    return forward_impl(h, x, ldx, y, ldy, B, dtype, flags, z_out, stream, false, nullptr);
}

extern "C" tsvd_status_t tsvd_forward_v(tsvd_handle_t h, const void* x, int ldx, float* t_out, int ldt, int B,
                                        tsvd_dtype_t dtype, unsigned flags, void* stream)
{
    if (!t_out) return TSVD_E_NULL;
    float* t = nullptr;
    const tsvd_status_t st = forward_impl(h, x, ldx, t_out, ldt, B, dtype, flags, nullptr, stream, true, &t);
    if (st != TSVD_OK) return st;
    // the stage wrote all padded rows into the handle's scratch: the K real ones go to the caller
    TSVD_CUDA_OK(cudaMemcpy2DAsync(t_out, (size_t)ldt * sizeof(float), t, (size_t)h->V.R_pad * sizeof(float),
                                   (size_t)h->K * sizeof(float), (size_t)B, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return TSVD_OK;
}

extern "C" tsvd_status_t tsvd_forward_v_patches(tsvd_handle_t h, const void* x, tsvd_dtype_t dtype, int n_img, int H, int W,
                                                int C, int k1, int k2, int stride_h, int stride_w, int pad_h, int pad_w,
                                                int dil_h, int dil_w, float* t_out, int ldt, unsigned flags, void* stream)
{
    if (!h || !x || !t_out) return TSVD_E_NULL;
    if (n_img < 1 || H < 1 || W < 1 || C < 1 || k1 < 1 || k2 < 1 || stride_h < 1 || stride_w < 1 || pad_h < 0 || pad_w < 0 ||
        dil_h < 1 || dil_w < 1)
        return TSVD_E_SHAPE;
    const int Ho = (H + 2 * pad_h - dil_h * (k1 - 1) - 1) / stride_h + 1;
    const int Wo = (W + 2 * pad_w - dil_w * (k2 - 1) - 1) / stride_w + 1;
    const long long feat = (long long)k1 * k2 * C, B = (long long)n_img * Ho * Wo;
    if (Ho < 1 || Wo < 1 || feat != h->N || B > 0x7fffffffLL || C % 16 != 0) return TSVD_E_SHAPE;
    PatchGather g;
    g.H = H; g.W = W; g.C = C; g.k2 = k2; g.sh = stride_h; g.sw = stride_w; g.ph = pad_h; g.pw = pad_w;
    g.dh = dil_h; g.dw = dil_w; g.Ho = Ho; g.Wo = Wo; g.feat = (int)feat;
    float* t = nullptr;
    const tsvd_status_t st = forward_impl(h, x, h->N, t_out, ldt, (int)B, dtype, flags, nullptr, stream, true, &t, &g);
    if (st != TSVD_OK) return st;
    TSVD_CUDA_OK(cudaMemcpy2DAsync(t_out, (size_t)ldt * sizeof(float), t, (size_t)h->V.R_pad * sizeof(float),
                                   (size_t)h->K * sizeof(float), (size_t)B, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return TSVD_OK;
}

// The largest scratch any path asks for with up to B_max tokens of this dtype: every path's need
// grows with the batch inside its own regime, so the regime boundaries and B_max cover it.
extern "C" tsvd_status_t tsvd_reserve(tsvd_handle_t h, int B_max, tsvd_dtype_t dtype)
{
    if (!h) return TSVD_E_NULL;
    if (B_max < 1) return TSVD_E_SHAPE;
    if (dtype_size(dtype) == 0) return TSVD_E_DTYPE;
    int dev = 0;
    TSVD_CUDA_OK(cudaGetDevice(&dev));
    if (dev != h->device) return TSVD_E_CUDA;
    size_t need = 0;
    for (int wide = 0; wide < 2; ++wide) {
        const size_t t = tsvd_tensor_ws_bytes_upto(h, B_max, dtype, wide != 0);
        if (t > need) need = t;
    }
    const int marks[] = {B_max, TSVD_DECODE_MAX_B, TSVD_INDEX_MAX_B};
    for (int B : marks) {
        if (B > B_max) continue;
        const size_t d = tsvd_decode_ws_bytes(h, B), s = tsvd_simple_ws_bytes(h, B);
        if (d > need) need = d;
        if (s > need) need = s;
    }
    return ensure_ws(h, need);
}

extern "C" tsvd_status_t tsvd_forward(tsvd_handle_t h, const void* x, void* y, int B, tsvd_dtype_t dtype,
                                      void* stream)
{
    if (!h) return TSVD_E_NULL;
    return tsvd_forward_ex(h, x, h->N, y, h->M, B, dtype, 0u, nullptr, stream);
}

// Host-buffer entry point.  The batch is cut into chunks of whole tiles and pipelined over three
// streams of the handle: the copy-in of chunk i+1 and the copy-out of chunk i-1 run while chunk i is
// computed (with pageable host memory the copies stage through the driver and overlap less).
static tsvd_status_t host_streams(tsvd_handle_s* h)
{
    for (int i = 0; i < 3; ++i)
        if (!h->host_stream[i]) TSVD_CUDA_OK(cudaStreamCreateWithFlags(&h->host_stream[i], cudaStreamNonBlocking));
    return TSVD_OK;
}

extern "C" tsvd_status_t tsvd_forward_host(tsvd_handle_t h, const void* x, void* y, int B,
                                           tsvd_dtype_t dtype, unsigned flags, void* z_out)
{
    if (!h || !x || !y) return TSVD_E_NULL;
    if (B < 1) return TSVD_E_SHAPE;
    const size_t xs = dtype_size(dtype);
    if (xs == 0) return TSVD_E_DTYPE;
    const bool y_bf16 = (dtype == TSVD_BF16) && !(flags & TSVD_FLAG_OUT_F32);
    const size_t ys = y_bf16 ? 2 : 4;
    const size_t x_bytes = (size_t)B * h->N * xs;
    const size_t y_bytes = (size_t)B * h->M * ys;
    const size_t z_bytes = z_out ? (size_t)B * h->K * 4 : 0;
    // staging buffers live in the handle and only grow
    const size_t x_off = 0, y_off = (x_bytes + 255) & ~(size_t)255;
    const size_t z_off = y_off + ((y_bytes + 255) & ~(size_t)255);
    const size_t need = z_off + z_bytes;
    if (need > h->io_bytes) {
        TSVD_CUDA_OK(cudaDeviceSynchronize());
        if (h->io) { cudaFree(h->io); h->io = nullptr; h->io_bytes = 0; }
        if (cudaMalloc(&h->io, need) != cudaSuccess) { (void)cudaGetLastError(); return TSVD_E_NOMEM; }
        h->io_bytes = need;
    }
    tsvd_status_t st = host_streams(h);
    if (st != TSVD_OK) return st;
    // chunks of whole tiles of both stages (64- and 48-token tiles: multiples of 192), about eight per
    // call, none below 384 tokens; small batches go in one piece
    int chunk = B;
    if (B >= 768) {
        chunk = ((B + 7) / 8 + 191) / 192 * 192;
        if (chunk < 384) chunk = 384;
    }
    const int n_chunks = (B + chunk - 1) / chunk;
    while ((int)h->host_events.size() < 2 * n_chunks) {
        cudaEvent_t e;
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) { (void)cudaGetLastError(); return TSVD_E_CUDA; }
        h->host_events.push_back(e);
    }
    char* base = reinterpret_cast<char*>(h->io);
    cudaStream_t s_in = h->host_stream[0], s_run = h->host_stream[1], s_out = h->host_stream[2];
    do {
        for (int c = 0; c < n_chunks && st == TSVD_OK; ++c) {
            const int b0 = c * chunk, nb = (B - b0 < chunk) ? B - b0 : chunk;
            const size_t xo = (size_t)b0 * h->N * xs, yo = (size_t)b0 * h->M * ys, zo = (size_t)b0 * h->K * 4;
            cudaEvent_t e_in = h->host_events[2 * c], e_run = h->host_events[2 * c + 1];
            if (cudaMemcpyAsync(base + x_off + xo, (const char*)x + xo, (size_t)nb * h->N * xs, cudaMemcpyHostToDevice, s_in) != cudaSuccess ||
                cudaEventRecord(e_in, s_in) != cudaSuccess || cudaStreamWaitEvent(s_run, e_in, 0) != cudaSuccess) { st = TSVD_E_CUDA; break; }
            st = tsvd_forward_ex(h, base + x_off + xo, h->N, base + y_off + yo, h->M, nb, dtype, flags,
                                 z_out ? base + z_off + zo : nullptr, s_run);
            if (st != TSVD_OK) break;
            if (cudaEventRecord(e_run, s_run) != cudaSuccess || cudaStreamWaitEvent(s_out, e_run, 0) != cudaSuccess) { st = TSVD_E_CUDA; break; }
            if (cudaMemcpyAsync((char*)y + yo, base + y_off + yo, (size_t)nb * h->M * ys, cudaMemcpyDeviceToHost, s_out) != cudaSuccess) { st = TSVD_E_CUDA; break; }
            if (z_out && cudaMemcpyAsync((char*)z_out + zo, base + z_off + zo, (size_t)nb * h->K * 4, cudaMemcpyDeviceToHost, s_out) != cudaSuccess) {
                st = TSVD_E_CUDA; break;
            }
        }
    } while (0);
    // everything queued so far is waited for, also after an error
    const cudaError_t e1 = cudaStreamSynchronize(s_in), e2 = cudaStreamSynchronize(s_run), e3 = cudaStreamSynchronize(s_out);
    if (st == TSVD_OK && (e1 != cudaSuccess || e2 != cudaSuccess || e3 != cudaSuccess)) st = TSVD_E_CUDA;
    if (st != TSVD_OK) (void)cudaGetLastError();
    return st;
}
