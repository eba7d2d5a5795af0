// pask_distortion: the inner term of the attention-output distortion of Eq. 4,
// max over query heads of || o_ref - o_test ||^2 for each decode position, from two attention
// outputs of this library (the full high-precision cache and a cache under some policy).
// Calibration-side consumer of the kernel pair; HBM-bound (reads both outputs once).
#include "pask_internal.h"

namespace pask {

namespace {

// One CTA per row (decode position), one warp per query head: 128 dims = 32 lanes x float4.
__global__ void __launch_bounds__(1024)
distortion_kernel(int n_rows, int n_q, const float4 *__restrict__ o_ref, const float4 *__restrict__ o_test,
                  float *__restrict__ per_row, double *__restrict__ sum) {
    __shared__ float s_head[32];
    const int row = blockIdx.x, lane = threadIdx.x & 31, head = threadIdx.x >> 5;
    const size_t at = ((size_t)row * n_q + head) * (kHeadDim / 4) + lane;
    const float4 a = o_ref[at], b = o_test[at];
    const float dx = a.x - b.x, dy = a.y - b.y, dz = a.z - b.z, dw = a.w - b.w;
    float d = dx * dx + dy * dy + dz * dz + dw * dw;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
    if (lane == 0) s_head[head] = d;
    __syncthreads();
    if (head == 0) {
        float m = lane < n_q ? s_head[lane] : 0.0f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0) {
            if (per_row) per_row[row] = m;
            if (sum) atomicAdd(sum, (double)m);
        }
    }
}

}  // namespace

}  // namespace pask

extern "C" pask_status_t pask_distortion(int32_t n_rows, int32_t n_q_heads, const float *o_ref, const float *o_test,
                                         float *per_row_out, double *sum_inout, pask_stream_t stream) {
    if (!o_ref || !o_test || n_rows < 0 || n_q_heads < 1 || n_q_heads > 32) return PASK_ERR_INVALID_ARG;
    if (((uintptr_t)o_ref | (uintptr_t)o_test) & 15 || ((uintptr_t)per_row_out & 3) || ((uintptr_t)sum_inout & 7))
        return PASK_ERR_INVALID_ARG;
    if (n_rows == 0) return PASK_OK;
    pask::distortion_kernel<<<n_rows, 32 * n_q_heads, 0, static_cast<cudaStream_t>(stream)>>>(
        n_rows, n_q_heads, reinterpret_cast<const float4 *>(o_ref), reinterpret_cast<const float4 *>(o_test), per_row_out,
        sum_inout);
    return cudaGetLastError() == cudaSuccess ? PASK_OK : PASK_ERR_CUDA;
}
