// Layer-wise top-k selection for one worker (Algorithm 5) as ONE persistent cooperative
// kernel: a segmented radix select over magnitude bit patterns followed by an ordered
// compaction.  One CTA of 512 threads per SM; five steps separated by grid barriers.  Every
// CTA owns the same tiles of the call in every step and keeps what it stages for them (in
// shared memory; overflow spills to HBM), so after the reading steps all work is local to the
// CTA that staged the data.
//
//   A   read 1: layers WITHOUT a remembered cut get a histogram of key bits 30..19 in shared memory,
//       flushed with integer atomics.  Layers WITH a speculative cut (predict_cut: where the previous
//       call found a key a little below the layer's k-th largest, moved by the change of the layer's
//       norm, lowered by how well that has been predicting) are not histogrammed element by element:
//       every entry at or above the cut is moved, in index order, behind the CTA's staging cursor and
//       counted under its bucket, which gives the complete histogram from the cut upwards.  The CTA
//       that flushes a layer's last tiles finds the bucket b1 holding the k-th largest key; a layer
//       whose counts do not reach k has its full histogram built in a second round of this step.
//   B   a CTA whose cuts were all at or below the true b1 already holds everything it needs
//       and reads nothing; any other CTA drops what it staged and reads its tiles a second
//       time with the true cut.  Then the staged entries of bucket b1 feed the level-2
//       histogram (bits 18..9).
//   S2  every CTA finds bucket b2 of its layers from the level-2 histograms, then adds the
//       level-3 histogram (bits 8..0) of its staged entries of bucket (b1, b2)
//   S3  every CTA fixes the exact threshold key T and the number of entries equal to T to
//       take, counts its staged entries above / equal to T per tile, publishes its totals
//   S4  every CTA adds up the totals of the tiles before its own, scans its own tiles, and
//       writes (value, int64 index) in ascending index (equal keys: lowest indices first);
//       optionally zeroes the selected entries of the vector (residual update)
// Layers of at most kDirectElems elements take no part in this: at the end one CTA loads
// each of them whole and finishes it from shared memory.
//
// The speculative cut only decides whether step B has to read: the staged set is always a
// superset of what the true cut keeps, so the result does not depend on it.  In a training
// loop the cut of a layer moves little from step to step and the vector is read once.
//
// Determinism: histograms use integer atomics (order-free); the staging order inside a CTA
// depends on warp timing but every output position is a function of counts and of the tile
// an entry came from, so the result is bit-identical from run to run.
#include "deft_select_steps.cuh"

namespace cg = cooperative_groups;

namespace deft {
namespace {

__global__ void __launch_bounds__(kSelThreads, 1) k_select_fused(const SelParams p_in) {
    extern __shared__ __align__(16) unsigned char smem[];
    cg::grid_group grid = cg::this_grid();
    const SelParams& p = params_in_smem(p_in, smem);
    if (p.timing && threadIdx.x == 0 && blockIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        p.timing[0] = t;
    }
    five_steps(p, smem, grid);
}

__global__ void k_zero_at(float* __restrict__ acc, const int64_t* __restrict__ idx, int64_t count) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count;
         i += (int64_t)gridDim.x * blockDim.x)
        acc[idx[i]] = 0.0f;
}

// CLT-k follower: own values at the leader's indices, then cleared.
__global__ void k_gather_zero(float* __restrict__ acc, const int64_t* __restrict__ idx, int64_t count,
                              float* __restrict__ val) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t j = idx[i];
        val[i] = acc[j];
        acc[j] = 0.0f;
    }
}

}  // namespace

deft_status launch_select(const SelParams& p, cudaStream_t stream) {
    static thread_local int attr_dev = -1;
    int dev = 0;
    DEFT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != attr_dev) {
        DEFT_CUDA_TRY(cudaFuncSetAttribute(k_select_fused, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           kSmemBytes));
        attr_dev = dev;
    }
    SelParams args = p;
    void* kargs[] = {&args};
    DEFT_CUDA_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(k_select_fused), dim3(p.grid),
                                              dim3(kSelThreads), kargs, kSmemBytes, stream));
    return DEFT_OK;
}

deft_status launch_residual_update(float* acc_d, const int64_t* idx_d, int64_t count,
                                   cudaStream_t stream) {
    if (count == 0) return DEFT_OK;
    const int64_t want = (count + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 16;
    k_zero_at<<<(int)(want < cap ? want : cap), 256, 0, stream>>>(acc_d, idx_d, count);
    DEFT_CUDA_TRY(cudaGetLastError());
    return DEFT_OK;
}

deft_status launch_gather_update(float* acc_d, const int64_t* idx_d, int64_t count, float* val_d,
                                 cudaStream_t stream) {
    if (count == 0) return DEFT_OK;
    const int64_t want = (count + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 16;
    k_gather_zero<<<(int)(want < cap ? want : cap), 256, 0, stream>>>(acc_d, idx_d, count, val_d);
    DEFT_CUDA_TRY(cudaGetLastError());
    return DEFT_OK;
}

}  // namespace deft
