// The pieces of Algorithm 1 around the sparsifier that a multi-worker run needs on the device:
// the union of the workers' index lists (line 7, after the all-gather), the sum and the average of
// the workers' contributions (lines 8-9 around the all-reduce), and the L2 norm of a whole vector
// (Eq. 2, the error).  Small kernels; none of them is on the selection's hot path.
#include "deft_common.cuh"

namespace deft {
namespace {

constexpr int kUThreads = 256;
constexpr int kUWordsPerThread = 4;
constexpr int kUWordsPerBlock = kUThreads * kUWordsPerThread;   // bitmap words (32 indices each) per block

__global__ void k_fill_start(int64_t* ls, int64_t n) {
    if (threadIdx.x == 0 && blockIdx.x == 0) { ls[0] = 0; ls[1] = n; }
}

__global__ void k_mark(const int64_t* __restrict__ idx, int64_t count, int64_t n, uint32_t* bitmap) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t v = idx[i];
        if (v >= 0 && v < n) atomicOr(bitmap + (v >> 5), 1u << (v & 31));
    }
}

// Set bits per block of kUWordsPerBlock bitmap words.
__global__ void __launch_bounds__(kUThreads) k_count_bits(const uint32_t* __restrict__ bitmap, int64_t words, uint32_t* block_sum) {
    __shared__ uint32_t sh[kUThreads / 32];
    const int64_t w0 = (int64_t)blockIdx.x * kUWordsPerBlock + (int64_t)threadIdx.x * kUWordsPerThread;
    uint32_t c = 0;
#pragma unroll
    for (int u = 0; u < kUWordsPerThread; ++u)
        if (w0 + u < words) c += __popc(bitmap[w0 + u]);
    c = __reduce_add_sync(0xffffffffu, c);
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t t = 0;
        for (int i = 0; i < kUThreads / 32; ++i) t += sh[i];
        block_sum[blockIdx.x] = t;
    }
}

// Exclusive prefix of the block sums in place (one block; the sums are few: words / 1024), total to *count_out.
__global__ void __launch_bounds__(1024) k_scan_blocks(uint32_t* block_sum, int64_t blocks, long long* count_out) {
    __shared__ unsigned long long warp_tot[32];
    __shared__ unsigned long long carry;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int64_t b0 = 0; b0 < blocks; b0 += 1024) {
        const int64_t b = b0 + threadIdx.x;
        const unsigned long long v = b < blocks ? block_sum[b] : 0ull;
        unsigned long long incl = v;
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long x = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += x;
        }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        unsigned long long before = carry;
        for (int w = 0; w < warp; ++w) before += warp_tot[w];
        // the output positions are 64-bit; a block's own offset is kept in two 32-bit halves
        if (b < blocks) {
            const unsigned long long ex = before + incl - v;
            block_sum[b] = (uint32_t)ex;                       // low half in place
            block_sum[blocks + b] = (uint32_t)(ex >> 32);      // high half behind the sums
        }
        __syncthreads();
        if (threadIdx.x == 1023) carry = before + incl;
        __syncthreads();
    }
    if (threadIdx.x == 0) *count_out = (long long)carry;
}

// Writes the set bits of the block's words as int64 indices, ascending, at the block's offset.
__global__ void __launch_bounds__(kUThreads) k_emit_bits(const uint32_t* __restrict__ bitmap, int64_t words, int64_t blocks,
                                                         const uint32_t* __restrict__ block_off, int64_t* out, int64_t cap) {
    __shared__ uint32_t sh[kUThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t w0 = (int64_t)blockIdx.x * kUWordsPerBlock + (int64_t)threadIdx.x * kUWordsPerThread;
    uint32_t word[kUWordsPerThread];
    uint32_t c = 0;
#pragma unroll
    for (int u = 0; u < kUWordsPerThread; ++u) {
        word[u] = w0 + u < words ? bitmap[w0 + u] : 0u;
        c += __popc(word[u]);
    }
    uint32_t incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t x = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += x;
    }
    if (lane == 31) sh[warp] = incl;
    __syncthreads();
    uint32_t before = 0;
    for (int w = 0; w < warp; ++w) before += sh[w];
    int64_t pos = (int64_t)(((unsigned long long)block_off[blocks + blockIdx.x] << 32) | block_off[blockIdx.x]) + before + incl - c;
#pragma unroll
    for (int u = 0; u < kUWordsPerThread; ++u) {
        uint32_t m = word[u];
        while (m) {
            const int bit = __ffs((int)m) - 1;
            m &= m - 1;
            if (pos < cap) out[pos] = (w0 + u) * 32 + bit;
            ++pos;
        }
    }
}

__global__ void k_sum_into(float* __restrict__ dst, const float* __restrict__ src, int64_t count) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
        dst[i] = __fadd_rn(dst[i], src[i]);
}

__global__ void k_divide(float* __restrict__ x, int64_t count, float by) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
        x[i] = __fdiv_rn(x[i], by);
}

inline int grid_for(int64_t count, int threads) {
    const int64_t want = (count + threads - 1) / threads;
    const int64_t cap = (int64_t)sm_count() * 16;
    return (int)(want < 1 ? 1 : (want < cap ? want : cap));
}

}  // namespace

size_t union_ws_bytes(int64_t n) {
    const int64_t words = (n + 31) / 32;
    const int64_t blocks = (words + kUWordsPerBlock - 1) / kUWordsPerBlock;
    return align_up(sizeof(uint32_t) * (size_t)words, 256) + align_up(sizeof(uint32_t) * 2 * (size_t)blocks, 256);
}

deft_status launch_index_union(const int64_t* idx_d, int64_t count, int64_t n, int64_t* out_d, int64_t out_cap,
                               long long* count_out_d, void* ws_d, cudaStream_t stream) {
    const int64_t words = (n + 31) / 32;
    const int64_t blocks = (words + kUWordsPerBlock - 1) / kUWordsPerBlock;
    uint32_t* bitmap = static_cast<uint32_t*>(ws_d);
    uint32_t* block_sum = reinterpret_cast<uint32_t*>(static_cast<char*>(ws_d) + align_up(sizeof(uint32_t) * (size_t)words, 256));
    DEFT_CUDA_TRY(cudaMemsetAsync(bitmap, 0, sizeof(uint32_t) * (size_t)words, stream));
    if (count > 0) k_mark<<<grid_for(count, 256), 256, 0, stream>>>(idx_d, count, n, bitmap);
    k_count_bits<<<(unsigned)blocks, kUThreads, 0, stream>>>(bitmap, words, block_sum);
    k_scan_blocks<<<1, 1024, 0, stream>>>(block_sum, blocks, count_out_d);
    k_emit_bits<<<(unsigned)blocks, kUThreads, 0, stream>>>(bitmap, words, blocks, block_sum, out_d, out_cap);
    DEFT_CUDA_TRY(cudaGetLastError());
    return DEFT_OK;
}

deft_status launch_sum_into(float* dst_d, const float* src_d, int64_t count, cudaStream_t stream) {
    if (count == 0) return DEFT_OK;
    k_sum_into<<<grid_for(count, 256), 256, 0, stream>>>(dst_d, src_d, count);
    DEFT_CUDA_TRY(cudaGetLastError());
    return DEFT_OK;
}

deft_status launch_divide(float* x_d, int64_t count, float by, cudaStream_t stream) {
    if (count == 0) return DEFT_OK;
    k_divide<<<grid_for(count, 256), 256, 0, stream>>>(x_d, count, by);
    DEFT_CUDA_TRY(cudaGetLastError());
    return DEFT_OK;
}

deft_status launch_fill_start(int64_t* ls_d, int64_t n, cudaStream_t stream) {
    k_fill_start<<<1, 32, 0, stream>>>(ls_d, n);
    DEFT_CUDA_TRY(cudaGetLastError());
    return DEFT_OK;
}

}  // namespace deft
