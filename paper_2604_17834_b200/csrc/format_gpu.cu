// GPU-side construction of the BCSR format (Sec. 2.3) from a CSR matrix that already lives in
// device memory: block mask and index (which (I, J) blocks hold a stored entry, block columns
// ascending inside a block-row) and value packing into zero-filled b x b tiles.  Same arrays,
// bit for bit, as the host builder in format.cpp.
//
// One CTA per block-row.  The entries of a block-row are one contiguous range of the CSR
// arrays (rows I*b .. I*b + b - 1), and its block columns are collected in a shared-memory
// bitmap of ceil(k / b) bits:
//   count pass   bitmap -> number of stored blocks of the block-row
//   scan         exclusive prefix sum over block-rows -> block_row_ptr
//   fill pass    bitmap again, prefix popcounts over its words -> block_col_idx (ascending by
//                construction) and the slot of every entry's block; values scattered into
//                blocks[slot][row in block][column in block]
// A bitmap needs 2 * ceil(k / b) / 8 bytes of shared memory (bits + word prefix), at most 200 KB:
// k / b <= 819,200.
//
// WCSR (window condensation of Sec. 2.3): every stored entry becomes the 64-bit key
// (window << 32 | column); a radix sort and a unique pass (CUB primitives) leave, window after
// window, the ascending union of each window's columns; counting keys per window and two prefix
// sums give window_row_ptr (lengths padded to b_col) and each window's place in the key list;
// window_col_idx is those columns over a -1 fill, and every value finds its condensed column by
// binary search in its window's list and goes straight into the packed tile layout.
#include <cub/cub.cuh>

#include <cstring>
#include <numeric>
#include <algorithm>

#include "format.h"
#include "kernels.h"
#include "spmm_b200.h"

namespace spmm {

namespace {

constexpr int kThreads = 256;

// Validation in two passes, so that the second one never reads past the arrays: once row_ptr is
// known to start at 0 and to be monotone, every position below row_ptr[m] lies inside col_idx.
__global__ void csr_check_rows_kernel(int64_t m, const int64_t* row_ptr, int* err) {
    if (blockIdx.x == 0 && threadIdx.x == 0 && row_ptr[0] != 0) atomicMin(err, SPMM_ERR_INVALID_ARG);
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < m;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x)
        if (row_ptr[i + 1] < row_ptr[i]) atomicMin(err, SPMM_ERR_INVALID_ARG);
}

__global__ void csr_check_cols_kernel(int64_t m, int64_t k, const int64_t* row_ptr, const int32_t* col_idx, int* err) {
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < m;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        int64_t prev = -1;
        for (int64_t p = row_ptr[i]; p < row_ptr[i + 1]; ++p) {
            const int64_t c = col_idx[p];
            if (c < 0 || c >= k) { atomicMin(err, SPMM_ERR_OUT_OF_RANGE); break; }
            if (c <= prev) { atomicMin(err, SPMM_ERR_UNSORTED); break; }
            prev = c;
        }
    }
}

// Shared-memory bitmap of the block columns of block-row I.
__device__ __forceinline__ void mark_block_columns(uint32_t* bits, int words, int64_t I, int64_t m, int b,
                                                   const int64_t* row_ptr, const int32_t* col_idx) {
    for (int w = threadIdx.x; w < words; w += blockDim.x) bits[w] = 0u;
    __syncthreads();
    const int64_t r1 = (I + 1) * b < m ? (I + 1) * b : m;
    const int64_t p0 = row_ptr[I * b], p1 = row_ptr[r1];
    for (int64_t p = p0 + threadIdx.x; p < p1; p += blockDim.x) {
        const int J = col_idx[p] / b;
        atomicOr(&bits[J >> 5], 1u << (J & 31));
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kThreads)
bcsr_count_kernel(int64_t m, int b, int words, const int64_t* row_ptr, const int32_t* col_idx, int32_t* counts) {
    extern __shared__ uint32_t smem[];
    __shared__ int total;
    if (threadIdx.x == 0) total = 0;
    mark_block_columns(smem, words, blockIdx.x, m, b, row_ptr, col_idx);
    int n = 0;
    for (int w = threadIdx.x; w < words; w += blockDim.x) n += __popc(smem[w]);
    for (int o = 16; o > 0; o >>= 1) n += __shfl_down_sync(0xffffffffu, n, o);
    if ((threadIdx.x & 31) == 0 && n) atomicAdd(&total, n);
    __syncthreads();
    if (threadIdx.x == 0) counts[blockIdx.x] = total;
}

// out[0] = 0, out[i + 1] = counts[0] + ... + counts[i]; *overflow set if the total passes int32.
__global__ void __launch_bounds__(1024)
exclusive_scan_kernel(const int32_t* counts, int64_t n, int32_t* out, int* overflow) {
    __shared__ long long warp_sum[32];
    __shared__ long long carry;
    if (threadIdx.x == 0) { carry = 0; out[0] = 0; }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int64_t base = 0; base < n; base += blockDim.x) {
        const int64_t i = base + threadIdx.x;
        long long v = i < n ? counts[i] : 0;
        long long x = v;
        for (int o = 1; o < 32; o <<= 1) {
            const long long y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        if (lane == 31) warp_sum[warp] = x;
        __syncthreads();
        if (warp == 0) {
            long long s = warp_sum[lane];
            for (int o = 1; o < 32; o <<= 1) {
                const long long y = __shfl_up_sync(0xffffffffu, s, o);
                if (lane >= o) s += y;
            }
            warp_sum[lane] = s;
        }
        __syncthreads();
        const long long incl = carry + (warp ? warp_sum[warp - 1] : 0) + x;
        if (i < n) {
            if (incl >= (1ll << 31)) *overflow = 1;
            out[i + 1] = static_cast<int32_t>(incl);
        }
        __syncthreads();
        if (threadIdx.x == blockDim.x - 1) carry = incl;
        __syncthreads();
    }
}

template <int ES>
__global__ void __launch_bounds__(kThreads)
bcsr_fill_kernel(int64_t m, int b, int words, const int64_t* row_ptr, const int32_t* col_idx, const uint8_t* vals,
                 const int32_t* block_row_ptr, int32_t* block_col_idx, uint8_t* blocks) {
    extern __shared__ uint32_t smem[];
    uint32_t* bits = smem;
    uint32_t* prefix = smem + words;         // set bits in the words before this one
    __shared__ int warp_sum[kThreads / 32];
    __shared__ int carry;
    const int64_t I = blockIdx.x;
    mark_block_columns(bits, words, I, m, b, row_ptr, col_idx);
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int base = 0; base < words; base += blockDim.x) {
        const int w = base + threadIdx.x;
        const int v = w < words ? __popc(bits[w]) : 0;
        int x = v;
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        if (lane == 31) warp_sum[warp] = x;
        __syncthreads();
        if (warp == 0 && lane < kThreads / 32) {
            int s = warp_sum[lane];
            for (int o = 1; o < kThreads / 32; o <<= 1) {
                const int y = __shfl_up_sync(0xffu, s, o);
                if (lane >= o) s += y;
            }
            warp_sum[lane] = s;
        }
        __syncthreads();
        const int incl = carry + (warp ? warp_sum[warp - 1] : 0) + x;
        if (w < words) prefix[w] = static_cast<uint32_t>(incl - v);
        __syncthreads();
        if (threadIdx.x == blockDim.x - 1) carry = incl;
        __syncthreads();
    }
    const int32_t slot0 = block_row_ptr[I];
    // block columns, ascending: word by word, bit by bit
    for (int w = threadIdx.x; w < words; w += blockDim.x) {
        uint32_t x = bits[w];
        int32_t pos = slot0 + static_cast<int32_t>(prefix[w]);
        while (x) {
            const int bit = __ffs(x) - 1;
            block_col_idx[pos++] = w * 32 + bit;
            x &= x - 1;
        }
    }
    // values: one warp per row of the block-row
    const int64_t r1 = (I + 1) * b < m ? (I + 1) * b : m;
    const size_t tile_bytes = static_cast<size_t>(b) * b * ES;
    for (int64_t i = I * b + warp; i < r1; i += kThreads / 32) {
        const int64_t p0 = row_ptr[i], p1 = row_ptr[i + 1];
        for (int64_t p = p0 + lane; p < p1; p += 32) {
            const int c = col_idx[p];
            const int J = c / b;
            const uint32_t below = bits[J >> 5] & ((1u << (J & 31)) - 1u);
            const size_t slot = static_cast<size_t>(slot0) + prefix[J >> 5] + __popc(below);
            uint8_t* dst = blocks + slot * tile_bytes + (static_cast<size_t>(i - I * b) * b + (c - J * b)) * ES;
            const uint8_t* src = vals + static_cast<size_t>(p) * ES;
            if constexpr (ES == 1) *dst = *src;
            else if constexpr (ES == 2) *reinterpret_cast<uint16_t*>(dst) = *reinterpret_cast<const uint16_t*>(src);
            else *reinterpret_cast<uint32_t*>(dst) = *reinterpret_cast<const uint32_t*>(src);
        }
    }
}

}  // namespace

void finish_bcsr_host(BcsrHost* out) {
    const int64_t nbr = out->nbr;
    std::vector<uint8_t> col_used(static_cast<size_t>(out->nbc), 0);
    for (int32_t J : out->block_col_idx) col_used[J] = 1;
    out->distinct_bcols = std::count(col_used.begin(), col_used.end(), uint8_t{1});
    out->row_order.resize(static_cast<size_t>(nbr));
    std::iota(out->row_order.begin(), out->row_order.end(), 0);
    std::stable_sort(out->row_order.begin(), out->row_order.end(), [&](int32_t x, int32_t y) {
        const int32_t lx = out->block_row_ptr[x + 1] - out->block_row_ptr[x];
        const int32_t ly = out->block_row_ptr[y + 1] - out->block_row_ptr[y];
        return lx > ly;
    });
    out->n_empty = 0;
    for (int64_t I = 0; I < nbr; ++I)
        if (out->block_row_ptr[I + 1] == out->block_row_ptr[I]) out->n_empty++;
}

// One thread per 16-byte piece of the stacked values: sub-block r of stacked block s is stored
// block src[s][r] (b x b, row-major) or zeros.
__global__ void bcsr_stack_kernel(const uint4* __restrict__ blocks, const int32_t* __restrict__ src, uint4* __restrict__ out,
                                  int R, int pieces_per_block, int64_t n_pieces) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n_pieces) return;
    const int64_t sub = i / pieces_per_block;          // = s * R + r
    const int piece = static_cast<int>(i % pieces_per_block);
    const int32_t p = __ldg(src + sub);
    out[i] = p >= 0 ? __ldg(blocks + static_cast<int64_t>(p) * pieces_per_block + piece) : make_uint4(0u, 0u, 0u, 0u);
    (void)R;
}

int stack_bcsr_device(const uint8_t* d_blocks, const BcsrStack& st, int b, int es, uint8_t** d_stacked) {
    *d_stacked = nullptr;
    if (st.ns == 0) return SPMM_OK;
    const int pieces = b * b * es / 16;
    const int64_t n_pieces = st.ns * st.R * pieces;
    int32_t* d_src = nullptr;
    if (cudaMalloc(reinterpret_cast<void**>(&d_src), st.src.size() * 4) != cudaSuccess) return SPMM_ERR_ALLOC;
    if (cudaMalloc(reinterpret_cast<void**>(d_stacked), static_cast<size_t>(n_pieces) * 16) != cudaSuccess) {
        cudaFree(d_src);
        return SPMM_ERR_ALLOC;
    }
    int rc = SPMM_OK;
    if (cudaMemcpy(d_src, st.src.data(), st.src.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess) rc = SPMM_ERR_CUDA;
    if (!rc) {
        const int threads = 256;
        const int64_t grid = (n_pieces + threads - 1) / threads;
        bcsr_stack_kernel<<<static_cast<unsigned>(grid), threads>>>(reinterpret_cast<const uint4*>(d_blocks), d_src,
                                                                   reinterpret_cast<uint4*>(*d_stacked), st.R, pieces, n_pieces);
        if (cudaGetLastError() != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) rc = SPMM_ERR_CUDA;
    }
    cudaFree(d_src);
    if (rc) { cudaFree(*d_stacked); *d_stacked = nullptr; }
    return rc;
}

int build_bcsr_device(int64_t m, int64_t k, const int64_t* d_row_ptr, const int32_t* d_col_idx, const uint8_t* d_vals,
                      int es, int b, cudaStream_t st, BcsrHost* out, int64_t* nnz_out, int32_t** d_block_row_ptr,
                      int32_t** d_block_col_idx, uint8_t** d_blocks) {
    if (b != 16 && b != 32 && b != 64 && b != 128) return SPMM_ERR_UNSUPPORTED;
    if (es != 1 && es != 2 && es != 4) return SPMM_ERR_UNSUPPORTED;
    if (m < 0 || k < 0 || !d_row_ptr) return SPMM_ERR_INVALID_ARG;
    const int64_t nbr = (m + b - 1) / b, nbc = (k + b - 1) / b;
    const int words = static_cast<int>((nbc + 31) / 32);
    const size_t smem = static_cast<size_t>(2) * (words > 0 ? words : 1) * 4;
    if (smem > 200 * 1024) return SPMM_ERR_TOO_LARGE;
    *d_block_row_ptr = nullptr;
    *d_block_col_idx = nullptr;
    *d_blocks = nullptr;
    out->b = b;
    out->nbr = nbr;
    out->nbc = nbc;

    int* d_flags = nullptr;                     // [0] CSR error code (min), [1] scan overflow
    int32_t* d_counts = nullptr;
    auto fail = [&](int code) {
        cudaFree(d_flags);
        cudaFree(d_counts);
        cudaFree(*d_block_row_ptr);
        cudaFree(*d_block_col_idx);
        cudaFree(*d_blocks);
        *d_block_row_ptr = nullptr;
        *d_block_col_idx = nullptr;
        *d_blocks = nullptr;
        return code;
    };
    if (cudaMalloc(reinterpret_cast<void**>(&d_flags), 2 * sizeof(int)) != cudaSuccess) return fail(SPMM_ERR_ALLOC);
    if (cudaMemsetAsync(d_flags, 0, 2 * sizeof(int), st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
    if (cudaMalloc(reinterpret_cast<void**>(&d_counts), static_cast<size_t>(nbr + 1) * 4) != cudaSuccess) return fail(SPMM_ERR_ALLOC);
    if (cudaMalloc(reinterpret_cast<void**>(d_block_row_ptr), static_cast<size_t>(nbr + 1) * 4) != cudaSuccess) return fail(SPMM_ERR_ALLOC);

    // 1. the CSR must be canonical (the count and fill passes rely on in-range columns)
    int64_t nnz = 0;
    int flags[2] = {0, 0};
    const unsigned check_grid = static_cast<unsigned>(std::min<int64_t>((m + 255) / 256, 2048));
    if (m > 0) {
        csr_check_rows_kernel<<<check_grid, 256, 0, st>>>(m, d_row_ptr, d_flags);
        if (cudaMemcpyAsync(&nnz, d_row_ptr + m, sizeof(int64_t), cudaMemcpyDeviceToHost, st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
    }
    if (cudaMemcpyAsync(flags, d_flags, sizeof(flags), cudaMemcpyDeviceToHost, st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
    if (cudaStreamSynchronize(st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
    if (flags[0] != 0) return fail(flags[0]);
    if (nnz < 0 || (nnz > 0 && (!d_col_idx || !d_vals))) return fail(SPMM_ERR_INVALID_ARG);
    if (nnz > 0) {
        csr_check_cols_kernel<<<check_grid, 256, 0, st>>>(m, k, d_row_ptr, d_col_idx, d_flags);
        if (cudaMemcpyAsync(flags, d_flags, sizeof(flags), cudaMemcpyDeviceToHost, st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
        if (cudaStreamSynchronize(st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
        if (flags[0] != 0) return fail(flags[0]);
    }
    *nnz_out = nnz;

    // 2. stored blocks per block-row, 3. block_row_ptr
    if (smem > 48 * 1024) {
        cudaFuncSetAttribute(bcsr_count_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        cudaFuncSetAttribute(bcsr_fill_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        cudaFuncSetAttribute(bcsr_fill_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    }
    if (nbr > 0) bcsr_count_kernel<<<static_cast<unsigned>(nbr), kThreads, smem, st>>>(m, b, words, d_row_ptr, d_col_idx, d_counts);
    exclusive_scan_kernel<<<1, 1024, 0, st>>>(d_counts, nbr, *d_block_row_ptr, d_flags + 1);
    out->block_row_ptr.assign(static_cast<size_t>(nbr) + 1, 0);
    if (cudaMemcpyAsync(out->block_row_ptr.data(), *d_block_row_ptr, static_cast<size_t>(nbr + 1) * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return fail(SPMM_ERR_CUDA);
    if (cudaMemcpyAsync(flags, d_flags, sizeof(flags), cudaMemcpyDeviceToHost, st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
    if (cudaStreamSynchronize(st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
    if (flags[1]) return fail(SPMM_ERR_TOO_LARGE);
    const int64_t nnzb = out->block_row_ptr[static_cast<size_t>(nbr)];
    out->nnzb = nnzb;

    // 4. block columns and values
    const size_t tile_bytes = static_cast<size_t>(b) * b * es;
    const size_t idx_bytes = static_cast<size_t>(nnzb) * 4, val_bytes = static_cast<size_t>(nnzb) * tile_bytes;
    if (cudaMalloc(reinterpret_cast<void**>(d_block_col_idx), idx_bytes ? idx_bytes : 16) != cudaSuccess) return fail(SPMM_ERR_ALLOC);
    if (cudaMalloc(reinterpret_cast<void**>(d_blocks), val_bytes ? val_bytes : 16) != cudaSuccess) return fail(SPMM_ERR_ALLOC);
    if (val_bytes && cudaMemsetAsync(*d_blocks, 0, val_bytes, st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
    if (nbr > 0 && nnzb > 0) {
        if (es == 1)
            bcsr_fill_kernel<1><<<static_cast<unsigned>(nbr), kThreads, smem, st>>>(m, b, words, d_row_ptr, d_col_idx, d_vals, *d_block_row_ptr, *d_block_col_idx, *d_blocks);
        else if (es == 4)
            bcsr_fill_kernel<4><<<static_cast<unsigned>(nbr), kThreads, smem, st>>>(m, b, words, d_row_ptr, d_col_idx, d_vals, *d_block_row_ptr, *d_block_col_idx, *d_blocks);
        else
            bcsr_fill_kernel<2><<<static_cast<unsigned>(nbr), kThreads, smem, st>>>(m, b, words, d_row_ptr, d_col_idx, d_vals, *d_block_row_ptr, *d_block_col_idx, *d_blocks);
    }
    out->block_col_idx.assign(static_cast<size_t>(nnzb), 0);
    if (nnzb && cudaMemcpyAsync(out->block_col_idx.data(), *d_block_col_idx, idx_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return fail(SPMM_ERR_CUDA);
    if (cudaStreamSynchronize(st) != cudaSuccess || cudaGetLastError() != cudaSuccess) return fail(SPMM_ERR_CUDA);
    cudaFree(d_flags);
    cudaFree(d_counts);
    finish_bcsr_host(out);       // row order, empty block-rows, distinct block columns: host, from the index arrays
    return SPMM_OK;
}

namespace {

__global__ void wcsr_keys_kernel(int64_t m, int wh, const int64_t* row_ptr, const int32_t* col_idx, uint64_t* keys) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x) >> 5;
    const int64_t nwarps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    for (int64_t i = warp0; i < m; i += nwarps) {
        const uint64_t hi = static_cast<uint64_t>(i / wh) << 32;
        for (int64_t p = row_ptr[i] + lane; p < row_ptr[i + 1]; p += 32) keys[p] = hi | static_cast<uint32_t>(col_idx[p]);
    }
}

// per window: how many distinct columns; per column: is it referenced at all
__global__ void wcsr_count_kernel(const uint64_t* ukeys, const int* n_unique, int32_t* cnt, uint8_t* used) {
    const int64_t n = *n_unique;
    for (int64_t j = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; j < n;
         j += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const uint64_t key = ukeys[j];
        atomicAdd(&cnt[key >> 32], 1);
        used[static_cast<uint32_t>(key)] = 1;
    }
}

__global__ void wcsr_pad_kernel(const int32_t* cnt, int64_t nwin, int b_col, int32_t* len) {
    for (int64_t w = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; w < nwin;
         w += static_cast<int64_t>(gridDim.x) * blockDim.x)
        len[w] = (cnt[w] + b_col - 1) / b_col * b_col;
}

__global__ void wcsr_sum_used_kernel(const uint8_t* used, int64_t k, unsigned long long* total) {
    unsigned long long n = 0;
    for (int64_t c = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; c < k;
         c += static_cast<int64_t>(gridDim.x) * blockDim.x)
        n += used[c];
    for (int o = 16; o > 0; o >>= 1) n += __shfl_down_sync(0xffffffffu, n, o);
    if ((threadIdx.x & 31) == 0 && n) atomicAdd(total, n);
}

__global__ void wcsr_cols_kernel(const uint64_t* ukeys, const int* n_unique, const int32_t* ustart,
                                 const int32_t* window_row_ptr, int32_t* window_col_idx) {
    const int64_t n = *n_unique;
    for (int64_t j = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; j < n;
         j += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const uint64_t key = ukeys[j];
        const int64_t w = static_cast<int64_t>(key >> 32);
        window_col_idx[window_row_ptr[w] + (j - ustart[w])] = static_cast<int32_t>(static_cast<uint32_t>(key));
    }
}

template <int ES>
__global__ void wcsr_values_kernel(int64_t m, int wh, int b_col, const int64_t* row_ptr, const int32_t* col_idx,
                                   const uint8_t* vals, const int32_t* cnt, const int32_t* window_row_ptr,
                                   const int32_t* window_col_idx, uint8_t* packed) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x) >> 5;
    const int64_t nwarps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    for (int64_t i = warp0; i < m; i += nwarps) {
        const int64_t w = i / wh;
        const int r = static_cast<int>(i - w * wh);
        const int64_t base = window_row_ptr[w];
        const int32_t* seg = window_col_idx + base;
        const int n = cnt[w];
        for (int64_t p = row_ptr[i] + lane; p < row_ptr[i + 1]; p += 32) {
            const int32_t c = col_idx[p];
            int lo = 0, hi = n;                      // first position with seg[pos] >= c; c is in the list
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (seg[mid] < c) lo = mid + 1; else hi = mid;
            }
            uint8_t* dst = packed + wcsr_packed_offset(wh, b_col, ES, r, base + lo);
            const uint8_t* src = vals + static_cast<size_t>(p) * ES;
            if constexpr (ES == 1) *dst = *src;
            else if constexpr (ES == 2) *reinterpret_cast<uint16_t*>(dst) = *reinterpret_cast<const uint16_t*>(src);
            else *reinterpret_cast<uint32_t*>(dst) = *reinterpret_cast<const uint32_t*>(src);
        }
    }
}

// ---- reuse classes of the column groups (gather hints; the host rule of wcsr_reuse_classes)

__global__ void wcsr_refs_kernel(const int32_t* __restrict__ col_idx, int64_t P, int32_t* __restrict__ refs) {
    for (int64_t q = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; q < P; q += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int32_t c = col_idx[q];
        if (c >= 0) atomicAdd(refs + c, 1);
    }
}

__global__ void iota_kernel(int32_t* __restrict__ x, int64_t n) {
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += static_cast<int64_t>(gridDim.x) * blockDim.x)
        x[i] = static_cast<int32_t>(i);
}

// rows in descending order of their gather count (stable: ties by index): rank r -> class
__global__ void wcsr_class_kernel(const int32_t* __restrict__ sorted_refs, const int32_t* __restrict__ order, int64_t k,
                                  uint8_t* __restrict__ cls) {
    for (int64_t r = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; r < k; r += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        int level = 0;
        if (sorted_refs[r] > 1) {
            level = 7;
            for (int64_t lim = kWcsrTopClassRows; level > 0 && r >= lim; lim *= 2) --level;
        }
        cls[order[r]] = static_cast<uint8_t>(level);
    }
}

__global__ void wcsr_group_class_kernel(const int32_t* __restrict__ col_idx, int64_t n_groups, const uint8_t* __restrict__ cls,
                                        uint8_t* __restrict__ grp_class) {
    for (int64_t g = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; g < n_groups; g += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int4 c = reinterpret_cast<const int4*>(col_idx)[g];
        int best = 0;
        if (c.x >= 0) best = max(best, static_cast<int>(cls[c.x]));
        if (c.y >= 0) best = max(best, static_cast<int>(cls[c.y]));
        if (c.z >= 0) best = max(best, static_cast<int>(cls[c.z]));
        if (c.w >= 0) best = max(best, static_cast<int>(cls[c.w]));
        grp_class[g] = static_cast<uint8_t>(best);
    }
}

// Allocates and fills *d_grp_class [P / 4] from the device copy of window_col_idx.
int wcsr_reuse_classes_device(const int32_t* d_window_col_idx, int64_t P, int64_t k, cudaStream_t st, uint8_t** d_grp_class) {
    *d_grp_class = nullptr;
    if (P <= 0 || k <= 0) return SPMM_OK;
    int32_t *refs = nullptr, *refs_sorted = nullptr, *ids = nullptr, *order = nullptr;
    uint8_t* cls = nullptr;
    void* temp = nullptr;
    auto release = [&]() { cudaFree(refs); cudaFree(refs_sorted); cudaFree(ids); cudaFree(order); cudaFree(cls); cudaFree(temp); };
    const size_t kb = static_cast<size_t>(k) * 4;
    if (cudaMalloc(reinterpret_cast<void**>(&refs), kb) != cudaSuccess || cudaMalloc(reinterpret_cast<void**>(&refs_sorted), kb) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&ids), kb) != cudaSuccess || cudaMalloc(reinterpret_cast<void**>(&order), kb) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&cls), static_cast<size_t>(k)) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(d_grp_class), static_cast<size_t>(P / 4)) != cudaSuccess) {
        release();
        cudaFree(*d_grp_class);
        *d_grp_class = nullptr;
        return SPMM_ERR_ALLOC;
    }
    cudaMemsetAsync(refs, 0, kb, st);
    wcsr_refs_kernel<<<2048, 256, 0, st>>>(d_window_col_idx, P, refs);
    iota_kernel<<<static_cast<unsigned>(std::min<int64_t>((k + 255) / 256, 2048)), 256, 0, st>>>(ids, k);
    size_t tb = 0;
    cub::DeviceRadixSort::SortPairsDescending(nullptr, tb, refs, refs_sorted, ids, order, static_cast<int>(k), 0, 32, st);
    bool ok = cudaMalloc(&temp, tb ? tb : 16) == cudaSuccess &&
              cub::DeviceRadixSort::SortPairsDescending(temp, tb, refs, refs_sorted, ids, order, static_cast<int>(k), 0, 32, st) == cudaSuccess;
    if (ok) {
        wcsr_class_kernel<<<static_cast<unsigned>(std::min<int64_t>((k + 255) / 256, 2048)), 256, 0, st>>>(refs_sorted, order, k, cls);
        wcsr_group_class_kernel<<<2048, 256, 0, st>>>(d_window_col_idx, P / 4, cls, *d_grp_class);
        ok = cudaStreamSynchronize(st) == cudaSuccess && cudaGetLastError() == cudaSuccess;
    }
    release();
    if (!ok) {
        cudaFree(*d_grp_class);
        *d_grp_class = nullptr;
        return SPMM_ERR_CUDA;
    }
    return SPMM_OK;
}

}  // namespace

int build_wcsr_device(int64_t m, int64_t k, const int64_t* d_row_ptr, const int32_t* d_col_idx, const uint8_t* d_vals,
                      int es, int wh, int b_col, int T, int n_bins, cudaStream_t st, WcsrHost* out, int64_t* nnz_out,
                      int32_t** d_window_row_ptr, int32_t** d_window_col_idx, uint8_t** d_packed, uint8_t** d_grp_class) {
    *d_grp_class = nullptr;
    if (wh != 16 && wh != 64) return SPMM_ERR_UNSUPPORTED;
    if ((es != 1 && es != 2 && es != 4) || b_col * es != 32) return SPMM_ERR_UNSUPPORTED;
    if (T < 0 || T % b_col != 0 || n_bins <= 0) return SPMM_ERR_INVALID_ARG;
    if (m < 0 || k < 0 || !d_row_ptr) return SPMM_ERR_INVALID_ARG;
    const int64_t nwin = (m + wh - 1) / wh;
    out->wh = wh;
    out->b_col = b_col;
    out->nwin = nwin;
    *d_window_row_ptr = nullptr;
    *d_window_col_idx = nullptr;
    *d_packed = nullptr;

    int* d_flags = nullptr;                   // [0] CSR error code, [1] scan overflow, [2] number of unique keys
    uint64_t *d_keys = nullptr, *d_keys2 = nullptr;
    int32_t *d_cnt = nullptr, *d_len = nullptr, *d_ustart = nullptr;
    uint8_t* d_used = nullptr;
    unsigned long long* d_total = nullptr;
    void* d_temp = nullptr;
    auto release = [&]() {
        cudaFree(d_flags); cudaFree(d_keys); cudaFree(d_keys2); cudaFree(d_cnt); cudaFree(d_len);
        cudaFree(d_ustart); cudaFree(d_used); cudaFree(d_total); cudaFree(d_temp);
    };
    auto fail = [&](int code) {
        release();
        cudaFree(*d_window_row_ptr); cudaFree(*d_window_col_idx); cudaFree(*d_packed);
        *d_window_row_ptr = nullptr; *d_window_col_idx = nullptr; *d_packed = nullptr;
        return code;
    };
    auto alloc = [&](void** ptr, size_t bytes) { return cudaMalloc(ptr, bytes ? bytes : 16) == cudaSuccess; };

    if (!alloc(reinterpret_cast<void**>(&d_flags), 4 * sizeof(int))) return fail(SPMM_ERR_ALLOC);
    if (cudaMemsetAsync(d_flags, 0, 4 * sizeof(int), st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
    int64_t nnz = 0;
    int flags[4] = {0, 0, 0, 0};
    const unsigned check_grid = static_cast<unsigned>(std::min<int64_t>((m + 255) / 256, 2048));
    if (m > 0) {
        csr_check_rows_kernel<<<check_grid, 256, 0, st>>>(m, d_row_ptr, d_flags);
        if (cudaMemcpyAsync(&nnz, d_row_ptr + m, sizeof(int64_t), cudaMemcpyDeviceToHost, st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
    }
    if (cudaMemcpyAsync(flags, d_flags, sizeof(flags), cudaMemcpyDeviceToHost, st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
    if (cudaStreamSynchronize(st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
    if (flags[0] != 0) return fail(flags[0]);
    if (nnz < 0 || (nnz > 0 && (!d_col_idx || !d_vals))) return fail(SPMM_ERR_INVALID_ARG);
    if (nnz >= (int64_t{1} << 31)) return fail(SPMM_ERR_TOO_LARGE);
    if (nnz > 0) {
        csr_check_cols_kernel<<<check_grid, 256, 0, st>>>(m, k, d_row_ptr, d_col_idx, d_flags);
        if (cudaMemcpyAsync(flags, d_flags, sizeof(flags), cudaMemcpyDeviceToHost, st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
        if (cudaStreamSynchronize(st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
        if (flags[0] != 0) return fail(flags[0]);
    }
    *nnz_out = nnz;

    // keys -> sorted -> unique
    if (!alloc(reinterpret_cast<void**>(&d_keys), static_cast<size_t>(nnz) * 8) ||
        !alloc(reinterpret_cast<void**>(&d_keys2), static_cast<size_t>(nnz) * 8) ||
        !alloc(reinterpret_cast<void**>(&d_cnt), static_cast<size_t>(nwin + 1) * 4) ||
        !alloc(reinterpret_cast<void**>(&d_len), static_cast<size_t>(nwin + 1) * 4) ||
        !alloc(reinterpret_cast<void**>(&d_ustart), static_cast<size_t>(nwin + 1) * 4) ||
        !alloc(reinterpret_cast<void**>(&d_used), static_cast<size_t>(k)) ||
        !alloc(reinterpret_cast<void**>(&d_total), 8) ||
        !alloc(reinterpret_cast<void**>(d_window_row_ptr), static_cast<size_t>(nwin + 1) * 4))
        return fail(SPMM_ERR_ALLOC);
    cudaMemsetAsync(d_cnt, 0, static_cast<size_t>(nwin + 1) * 4, st);
    cudaMemsetAsync(d_used, 0, static_cast<size_t>(k ? k : 1), st);
    cudaMemsetAsync(d_total, 0, 8, st);
    const int n = static_cast<int>(nnz);
    int end_bit = 32;
    while (end_bit < 64 && (int64_t{1} << (end_bit - 32)) < nwin) ++end_bit;
    if (n > 0) {
        wcsr_keys_kernel<<<static_cast<unsigned>(std::min<int64_t>((m + 7) / 8, 4096)), 256, 0, st>>>(m, wh, d_row_ptr, d_col_idx, d_keys);
        size_t t1 = 0, t2 = 0;
        cub::DeviceRadixSort::SortKeys(nullptr, t1, d_keys, d_keys2, n, 0, end_bit, st);
        cub::DeviceSelect::Unique(nullptr, t2, d_keys2, d_keys, d_flags + 2, n, st);
        if (!alloc(&d_temp, std::max(t1, t2))) return fail(SPMM_ERR_ALLOC);
        size_t tb = std::max(t1, t2);
        if (cub::DeviceRadixSort::SortKeys(d_temp, tb, d_keys, d_keys2, n, 0, end_bit, st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
        tb = std::max(t1, t2);
        if (cub::DeviceSelect::Unique(d_temp, tb, d_keys2, d_keys, d_flags + 2, n, st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
        // d_keys now holds the unique keys, d_flags[2] their number
        wcsr_count_kernel<<<2048, 256, 0, st>>>(d_keys, d_flags + 2, d_cnt, d_used);
    }
    wcsr_pad_kernel<<<static_cast<unsigned>(std::min<int64_t>((nwin + 255) / 256 + 1, 2048)), 256, 0, st>>>(d_cnt, nwin, b_col, d_len);
    exclusive_scan_kernel<<<1, 1024, 0, st>>>(d_len, nwin, *d_window_row_ptr, d_flags + 1);
    exclusive_scan_kernel<<<1, 1024, 0, st>>>(d_cnt, nwin, d_ustart, d_flags + 3);
    if (k > 0) wcsr_sum_used_kernel<<<static_cast<unsigned>(std::min<int64_t>((k + 255) / 256, 1024)), 256, 0, st>>>(d_used, k, d_total);
    out->window_row_ptr.assign(static_cast<size_t>(nwin) + 1, 0);
    unsigned long long distinct = 0;
    if (cudaMemcpyAsync(out->window_row_ptr.data(), *d_window_row_ptr, static_cast<size_t>(nwin + 1) * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemcpyAsync(flags, d_flags, sizeof(flags), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemcpyAsync(&distinct, d_total, 8, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return fail(SPMM_ERR_CUDA);
    if (cudaStreamSynchronize(st) != cudaSuccess) return fail(SPMM_ERR_CUDA);
    if (flags[1]) return fail(SPMM_ERR_TOO_LARGE);
    const int64_t P = out->window_row_ptr[static_cast<size_t>(nwin)];
    out->P = P;
    out->distinct_cols = static_cast<int64_t>(distinct);

    // window_col_idx over a -1 fill, values into the zero-filled packed tiles
    const size_t packed_bytes = static_cast<size_t>(P) * wh * es;
    if (!alloc(reinterpret_cast<void**>(d_window_col_idx), static_cast<size_t>(P) * 4) ||
        !alloc(reinterpret_cast<void**>(d_packed), packed_bytes))
        return fail(SPMM_ERR_ALLOC);
    if (P > 0) {
        cudaMemsetAsync(*d_window_col_idx, 0xFF, static_cast<size_t>(P) * 4, st);
        cudaMemsetAsync(*d_packed, 0, packed_bytes, st);
    }
    if (n > 0) {
        wcsr_cols_kernel<<<2048, 256, 0, st>>>(d_keys, d_flags + 2, d_ustart, *d_window_row_ptr, *d_window_col_idx);
        const unsigned vgrid = static_cast<unsigned>(std::min<int64_t>((m + 7) / 8, 8192));
        if (es == 1)
            wcsr_values_kernel<1><<<vgrid, 256, 0, st>>>(m, wh, b_col, d_row_ptr, d_col_idx, d_vals, d_cnt, *d_window_row_ptr, *d_window_col_idx, *d_packed);
        else if (es == 2)
            wcsr_values_kernel<2><<<vgrid, 256, 0, st>>>(m, wh, b_col, d_row_ptr, d_col_idx, d_vals, d_cnt, *d_window_row_ptr, *d_window_col_idx, *d_packed);
        else
            wcsr_values_kernel<4><<<vgrid, 256, 0, st>>>(m, wh, b_col, d_row_ptr, d_col_idx, d_vals, d_cnt, *d_window_row_ptr, *d_window_col_idx, *d_packed);
    }
    if (cudaStreamSynchronize(st) != cudaSuccess || cudaGetLastError() != cudaSuccess) return fail(SPMM_ERR_CUDA);
    release();
    int rc = wcsr_reuse_classes_device(*d_window_col_idx, P, k, st, d_grp_class);
    if (!rc) rc = plan_wcsr(out, T, n_bins, es);
    if (rc) {
        cudaFree(*d_window_row_ptr); cudaFree(*d_window_col_idx); cudaFree(*d_packed); cudaFree(*d_grp_class);
        *d_window_row_ptr = nullptr; *d_window_col_idx = nullptr; *d_packed = nullptr; *d_grp_class = nullptr;
    }
    return rc;
}

}  // namespace spmm
