// Error-feedback accumulate fused with segmented per-layer sums of squares
// (Algorithm 1 line 5 + the per-layer gradient norm of Section 4.2).
//
// One streaming pass: 8 B read + 4 B written per element.  The vector is cut into
// address-aligned tiles of kTileA elements; a tile that lies inside one layer takes the
// vectorised path, a tile that crosses layer boundaries is processed piece by piece.
// Every (tile, layer) piece owns the partial-sum slot `tile + layer`, which is unique
// because both numbers only grow along the vector, so no atomics and no zero-fill are
// needed and the result is bit-identical from run to run.
#include "deft_common.cuh"

namespace deft {
namespace {

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum over the CTA in a fixed order; the result is valid in thread 0.
__device__ __forceinline__ double block_sum(double v, double* sh) {
    v = warp_sum(v);
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();  // sh may still be read from the previous use
    if (lane == 0) sh[w] = v;
    __syncthreads();
    double t = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int i = 0; i < kNormWarps; ++i) t += sh[i];
    }
    return t;
}

// Largest l in [0, L-1] with layer_start[l] <= pos.
__device__ __forceinline__ int layer_of(const int64_t* __restrict__ ls, int L, int64_t pos) {
    int lo = 0, hi = L - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (__ldg(ls + mid) <= pos) lo = mid; else hi = mid - 1;
    }
    return lo;
}

template <bool kHasGrad>
__global__ void __launch_bounds__(kNormThreads)
k_accum_norms(float* __restrict__ e, const float* __restrict__ g, int64_t n,
              const int64_t* __restrict__ ls, int L, double* __restrict__ partial, int64_t tiles) {
    __shared__ double sh[kNormWarps];
    for (int64_t t = blockIdx.x; t < tiles; t += gridDim.x) {
        const int64_t lo = t * kTileA;
        const int64_t hi = (lo + kTileA < n) ? lo + kTileA : n;
        int l = layer_of(ls, L, lo);
        if (hi - lo == kTileA && __ldg(ls + l + 1) >= hi) {
            // whole tile inside layer l: 8 float4 per thread, squares in fp32 per 8 elements
            float4* e4 = reinterpret_cast<float4*>(e + lo);
            const float4* g4 = reinterpret_cast<const float4*>(g + lo);
            double acc = 0.0;
#pragma unroll
            for (int i = 0; i < kTileA / (kNormThreads * 4); i += 2) {
                const int a = i * kNormThreads + threadIdx.x, b = a + kNormThreads;
                float4 x = e4[a], y = e4[b];
                if (kHasGrad) {
                    const float4 gx = __ldg(g4 + a), gy = __ldg(g4 + b);
                    x.x = __fadd_rn(x.x, gx.x); x.y = __fadd_rn(x.y, gx.y);
                    x.z = __fadd_rn(x.z, gx.z); x.w = __fadd_rn(x.w, gx.w);
                    y.x = __fadd_rn(y.x, gy.x); y.y = __fadd_rn(y.y, gy.y);
                    y.z = __fadd_rn(y.z, gy.z); y.w = __fadd_rn(y.w, gy.w);
                    e4[a] = x;
                    e4[b] = y;
                }
                float s = x.x * x.x;
                s = fmaf(x.y, x.y, s); s = fmaf(x.z, x.z, s); s = fmaf(x.w, x.w, s);
                s = fmaf(y.x, y.x, s); s = fmaf(y.y, y.y, s); s = fmaf(y.z, y.z, s);
                s = fmaf(y.w, y.w, s);
                acc += (double)s;
            }
            const double tot = block_sum(acc, sh);
            if (threadIdx.x == 0) partial[t + l] = tot;
        } else {
            // tile crosses layer boundaries (or is the ragged tail): one piece per layer
            int64_t ps = lo;
            while (ps < hi) {
                const int64_t lend = __ldg(ls + l + 1);
                const int64_t pe = lend < hi ? lend : hi;
                double acc = 0.0;
                for (int64_t i = ps + threadIdx.x; i < pe; i += kNormThreads) {
                    float x = e[i];
                    if (kHasGrad) {
                        x = __fadd_rn(x, __ldg(g + i));
                        e[i] = x;
                    }
                    acc += (double)x * (double)x;
                }
                const double tot = block_sum(acc, sh);
                if (threadIdx.x == 0 && pe > ps) partial[t + l] = tot;
                ps = pe;
                ++l;
            }
        }
    }
}

// One CTA per layer: add the layer's partial sums in a fixed order, take the root.
__global__ void __launch_bounds__(kNormThreads)
k_norm_finalize(const int64_t* __restrict__ ls, int L, const double* __restrict__ partial,
                double* __restrict__ norms, double* norms_host) {
    __shared__ double sh[kNormWarps];
    const int l = blockIdx.x;
    const int64_t s = ls[l], e = ls[l + 1];
    double acc = 0.0;
    if (e > s) {
        const int64_t t0 = s / kTileA, t1 = (e - 1) / kTileA;
        for (int64_t t = t0 + threadIdx.x; t <= t1; t += kNormThreads) acc += partial[t + l];
    }
    const double tot = block_sum(acc, sh);
    if (threadIdx.x == 0) {
        const double v = sqrt(tot);
        norms[l] = v;
        if (norms_host) {   // mapped host memory a waiting host thread polls: no stream synchronisation needed
            *reinterpret_cast<volatile double*>(norms_host + l) = v;
            __threadfence_system();
        }
    }
}

}  // namespace

deft_status launch_layer_norms(float* resid_acc_d, const float* grad_d, int64_t n_g,
                               const int64_t* layer_start_d, int32_t L, double* norms_d,
                               double* partial_d, cudaStream_t stream, double* norms_host_mapped) {
    const int64_t tiles = (n_g + kTileA - 1) / kTileA;
    // one CTA per tile: the hardware scheduler keeps the SMs evenly busy to the end, which a
    // resident grid-stride loop did not (0.645 -> 0.600 ms on 333.6 M elements); the loop in the
    // kernel only matters beyond 2^31 - 1 tiles
    const int64_t max_grid = 0x7fffffff;
    const int grid = (int)(tiles < max_grid ? tiles : max_grid);
    if (grad_d)
        k_accum_norms<true><<<grid, kNormThreads, 0, stream>>>(resid_acc_d, grad_d, n_g, layer_start_d,
                                                           L, partial_d, tiles);
    else
        k_accum_norms<false><<<grid, kNormThreads, 0, stream>>>(resid_acc_d, nullptr, n_g,
                                                            layer_start_d, L, partial_d, tiles);
    DEFT_CUDA_TRY(cudaGetLastError());
    k_norm_finalize<<<L, kNormThreads, 0, stream>>>(layer_start_d, L, partial_d, norms_d, norms_host_mapped);
    DEFT_CUDA_TRY(cudaGetLastError());
    return DEFT_OK;
}

}  // namespace deft
