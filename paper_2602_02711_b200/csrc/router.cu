// Inference-time calibration of the router (Sec. 4.2 "Inference-time calibration"): the threshold for a
// high-precision budget rho is the (1 - rho) quantile of the router's scores on a calibration pool,
//     tau(rho) = Quantile(D_cal, 1 - rho),
// and a step is served by the high-precision model when its score reaches the threshold, p_t >= tau.  The mask
// this writes is the one dmr_routed_linear reads, so scores go to a routed batch without leaving the device.
//
// Quantile rule (the paper names none): linear interpolation between order statistics, the common default -
// with the scores sorted ascending as x_(0) <= ... <= x_(n-1), h = (n - 1)(1 - rho), lo = floor(h),
// tau = x_(lo) + (h - lo) (x_(lo+1) - x_(lo)).  All of it in binary64 with every operation rounded on its own,
// so that the comparison p_t >= tau decides exactly as a plain CPU evaluation of the same formula does.
//
// Order statistics by counting: the rank of x_i is the number of elements that sort before it (ties broken by
// index, so ranks are unique); the two elements whose ranks are lo and lo + 1 are written out.  O(n^2)
// comparisons on n <= 65536 scores (the paper's pool: 64 tasks of at most 50 steps).
#include "common.cuh"

namespace dmr {

namespace {

constexpr int kRankThreads = 256;

__global__ void __launch_bounds__(kRankThreads) quantile_select_kernel(const float *__restrict__ x, int n, int lo, int hi,
                                                                       double *__restrict__ picked /*[2]*/) {
    __shared__ float tile[kRankThreads];
    const int i = blockIdx.x * kRankThreads + threadIdx.x;
    const float xi = i < n ? x[i] : 0.f;
    int rank = 0;
    for (int j0 = 0; j0 < n; j0 += kRankThreads) {
        const int j = j0 + threadIdx.x;
        tile[threadIdx.x] = j < n ? x[j] : 0.f;
        __syncthreads();
        const int m = min(kRankThreads, n - j0);
        for (int u = 0; u < m; ++u) {
            const float xj = tile[u];
            rank += (xj < xi || (xj == xi && j0 + u < i)) ? 1 : 0;
        }
        __syncthreads();
    }
    if (i < n) {
        if (rank == lo) picked[0] = (double)xi;
        if (rank == hi) picked[1] = (double)xi;
    }
}

__global__ void quantile_finish_kernel(const double *__restrict__ picked, double gamma, double *__restrict__ tau) {
    // x_lo + gamma (x_hi - x_lo), each operation rounded on its own (no fused multiply-add)
    *tau = __dadd_rn(picked[0], __dmul_rn(gamma, __dsub_rn(picked[1], picked[0])));
}

__global__ void router_mask_kernel(const float *__restrict__ p, int M, const double *__restrict__ tau, uint8_t *__restrict__ mask) {
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m < M) mask[m] = (double)p[m] >= *tau ? 1 : 0;
}

}  // namespace

dmr_status_t launch_router_calibrate(const float *scores, int n, double rho, double *tau, double *picked, cudaStream_t st) {
    const double h = (double)(n - 1) * (1.0 - rho);
    int lo = (int)h;  // h >= 0
    if (lo > n - 1) lo = n - 1;
    const int hi = lo + 1 < n ? lo + 1 : lo;
    const double gamma = h - (double)lo;
    quantile_select_kernel<<<(n + kRankThreads - 1) / kRankThreads, kRankThreads, 0, st>>>(scores, n, lo, hi, picked);
    dmr_status_t r = check_launch();
    if (r != DMR_OK) return r;
    quantile_finish_kernel<<<1, 1, 0, st>>>(picked, gamma, tau);
    return check_launch();
}

dmr_status_t launch_router_mask(const float *scores, int M, const double *tau, uint8_t *mask, cudaStream_t st) {
    router_mask_kernel<<<(M + 255) / 256, 256, 0, st>>>(scores, M, tau, mask);
    return check_launch();
}

}  // namespace dmr
