// Packer: int8 ternary matrices -> 2-bit codes in the tiled layout of tsvd_internal.cuh,
// and its inverse for tests.  The paper states only the storage cost, two bits per entry
// of a ternary matrix (Section "Connection with BNN and What Next").
#include "tsvd_internal.cuh"

namespace {

// One thread builds one 32-bit word = 16 consecutive columns of one row.
// flag bit 0 is raised if any entry is outside {-1,0,+1}.
__global__ void pack_words_kernel(const int8_t* __restrict__ T, int R, int C, int R_pad, int C_pad,
                                  uint32_t* __restrict__ words, int* __restrict__ flag,
                                  unsigned long long* __restrict__ nnz)
{
    const int words_per_row = C_pad >> 4;
    const size_t total = (size_t)R_pad * words_per_row;
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    unsigned local_nnz = 0;
    bool bad = false;
    if (idx < total) {
        const int row = (int)(idx / words_per_row);
        const int wi = (int)(idx % words_per_row);
        uint32_t w = 0;
        if (row < R) {
            const int8_t* src = T + (size_t)row * C + (size_t)wi * 16;
            const int c0 = wi * 16;
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                int v = (c0 + e < C) ? (int)src[e] : 0;
                if (v < -1 || v > 1) bad = true;
                uint32_t code = (v != 0 ? 1u : 0u) | (v < 0 ? 2u : 0u);
                w |= code << tsvd_entry_shift(e);
                local_nnz += (v != 0);
            }
        }
        const size_t unit = tsvd_unit_index(row, wi >> 2, C_pad);
        words[unit * 4 + (wi & 3)] = w;
    }
    if (bad) atomicOr(flag, 1);
    // warp-level sum of the nonzero count, one atomic per warp
    for (int o = 16; o > 0; o >>= 1) local_nnz += __shfl_down_sync(0xffffffffu, local_nnz, o);
    if ((threadIdx.x & 31) == 0 && local_nnz) atomicAdd(nnz, (unsigned long long)local_nnz);
}

__global__ void unpack_words_kernel(const uint32_t* __restrict__ words, int R, int C, int C_pad,
                                    int8_t* __restrict__ T)
{
    const int words_per_row = C_pad >> 4;
    const size_t total = (size_t)R * words_per_row;
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int row = (int)(idx / words_per_row);
    const int wi = (int)(idx % words_per_row);
    const size_t unit = tsvd_unit_index(row, wi >> 2, C_pad);
    const uint32_t w = words[unit * 4 + (wi & 3)];
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        const int c = wi * 16 + e;
        if (c < C) {
            const uint32_t code = (w >> tsvd_entry_shift(e)) & 3u;
            T[(size_t)row * C + c] = (int8_t)((code & 1u) ? ((code & 2u) ? -1 : 1) : 0);
        }
    }
}

inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

}  // namespace

tsvd_status_t tsvd_pack_matrix(const int8_t* host, int R, int C, PackedMat* out, int* dev_flag)
{
    PackedMat pm;
    pm.R = R;
    pm.C = C;
    pm.R_pad = round_up(R, TSVD_ROW_TILE);
    pm.C_pad = round_up(C, TSVD_COL_PAD);
    pm.n_units = (size_t)pm.R_pad * (size_t)(pm.C_pad / TSVD_COL_GROUP);

    int8_t* d_src = nullptr;
    unsigned long long* d_nnz = nullptr;
    const size_t src_bytes = (size_t)R * (size_t)C;
    cudaError_t e = cudaMalloc(&d_src, src_bytes);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return TSVD_E_NOMEM; }
    e = cudaMalloc(&pm.units, pm.bytes());
    if (e != cudaSuccess) { (void)cudaGetLastError(); cudaFree(d_src); return TSVD_E_NOMEM; }
    e = cudaMalloc(&d_nnz, sizeof(unsigned long long));
    if (e != cudaSuccess) { (void)cudaGetLastError(); cudaFree(d_src); cudaFree(pm.units); return TSVD_E_NOMEM; }

    tsvd_status_t st = TSVD_OK;
    do {
        if (cudaMemcpy(d_src, host, src_bytes, cudaMemcpyHostToDevice) != cudaSuccess) { st = TSVD_E_CUDA; break; }
        if (cudaMemset(d_nnz, 0, sizeof(unsigned long long)) != cudaSuccess) { st = TSVD_E_CUDA; break; }
        const size_t total = (size_t)pm.R_pad * (size_t)(pm.C_pad / 16);
        const int threads = 256;
        const unsigned blocks = (unsigned)((total + threads - 1) / threads);
        pack_words_kernel<<<blocks, threads>>>(d_src, R, C, pm.R_pad, pm.C_pad,
                                               reinterpret_cast<uint32_t*>(pm.units), dev_flag, d_nnz);
        tsvd_count_launch();
        if (cudaGetLastError() != cudaSuccess) { st = TSVD_E_CUDA; break; }
        if (cudaMemcpy(&pm.nnz, d_nnz, sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess) {
            st = TSVD_E_CUDA;
            break;
        }
    } while (0);
    cudaFree(d_src);
    cudaFree(d_nnz);
    if (st != TSVD_OK) {
        (void)cudaGetLastError();
        cudaFree(pm.units);
        return st;
    }
    *out = pm;
    return TSVD_OK;
}

tsvd_status_t tsvd_unpack_matrix(const PackedMat& pm, int8_t* host)
{
    int8_t* d_dst = nullptr;
    const size_t bytes = (size_t)pm.R * (size_t)pm.C;
    if (cudaMalloc(&d_dst, bytes) != cudaSuccess) { (void)cudaGetLastError(); return TSVD_E_NOMEM; }
    const size_t total = (size_t)pm.R * (size_t)(pm.C_pad / 16);
    const int threads = 256;
    const unsigned blocks = (unsigned)((total + threads - 1) / threads);
    unpack_words_kernel<<<blocks, threads>>>(reinterpret_cast<const uint32_t*>(pm.units), pm.R, pm.C,
                                             pm.C_pad, d_dst);
    tsvd_count_launch();
    tsvd_status_t st = TSVD_OK;
    if (cudaGetLastError() != cudaSuccess) st = TSVD_E_CUDA;
    if (st == TSVD_OK && cudaMemcpy(host, d_dst, bytes, cudaMemcpyDeviceToHost) != cudaSuccess) st = TSVD_E_CUDA;
    cudaFree(d_dst);
    if (st != TSVD_OK) (void)cudaGetLastError();
    return st;
}
