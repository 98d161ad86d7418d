// Route partition: the per-step precision decision r_t (Sec. 3, Eq. 1) arrives as a byte mask,
// 1 = the step needs the high-precision weights (Sec. 4.2, "KL-to-Classification Mapping").
// A stable partition turns it into two ascending row lists, so that each precision's rows can be
// multiplied as one dense batch and written back at their own positions (step order).
#include "sm100.cuh"

namespace dmr {

namespace {

constexpr int kPartThreads = 1024;

// One CTA walks the mask in chunks of 1024 rows; ballots and a 32-entry scan keep the order stable.
__global__ void __launch_bounds__(kPartThreads)
route_partition_kernel(const uint8_t *__restrict__ mask, int M, int32_t *__restrict__ idx_high,
                       int32_t *__restrict__ idx_low, int32_t *__restrict__ counts) {
    __shared__ int warp_high[32];
    __shared__ int base_high_s, base_low_s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    pdl_wait();  // the lists may still be read, and the mask written, by kernels before this one
    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        base_high_s = 0;
        base_low_s = 0;
    }
    __syncthreads();
    for (int m0 = 0; m0 < M; m0 += kPartThreads) {
        const int m = m0 + threadIdx.x;
        const bool valid = m < M;
        const bool high = valid && mask[m] != 0;
        const unsigned bh = __ballot_sync(0xFFFFFFFFu, high);
        if (lane == 0) warp_high[warp] = __popc(bh);
        __syncthreads();
        int before = 0, total_high = 0;  // high rows in earlier warps of this chunk / in the chunk
        for (int w = 0; w < 32; ++w) {
            const int c = warp_high[w];
            if (w < warp) before += c;
            total_high += c;
        }
        const int chunk_rows = min(kPartThreads, M - m0);
        const int high_rank = before + __popc(bh & ((1u << lane) - 1u));
        const int low_rank = threadIdx.x - high_rank;  // rows before me that are not high
        const int bh0 = base_high_s, bl0 = base_low_s;
        if (valid) {
            if (high) idx_high[bh0 + high_rank] = m;
            else idx_low[bl0 + low_rank] = m;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            base_high_s = bh0 + total_high;
            base_low_s = bl0 + (chunk_rows - total_high);
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        counts[0] = base_high_s;
        counts[1] = base_low_s;
    }
}

}  // namespace

dmr_status_t launch_route_partition(const uint8_t *mask, int M, int32_t *idx_high, int32_t *idx_low,
                                    int32_t *counts, cudaStream_t st) {
    (void)launch_pdl(route_partition_kernel, dim3(1), dim3(kPartThreads), 0, st, mask, M, idx_high, idx_low, counts);
    return check_launch();
}

}  // namespace dmr
