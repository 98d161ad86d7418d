// Any-shape fallback linear layers (CUDA cores): shapes the streaming and tensor-core kernels do not
// take, e.g. K that is not a multiple of the quantization unit they consume.
#include <cuda_bf16.h>

#include "common.cuh"

namespace dmr {

namespace {

// ---------------------------------------------------------------------------------------------
// Any-shape fallback: one warp per output feature, fp32 FMAs, lanes stride over k in chunks of 8.
// ---------------------------------------------------------------------------------------------
template <int MODE /*0 dense, 3, 4, 8*/, bool OUT_F32>
__global__ void __launch_bounds__(256)
simple_linear_kernel(const uint16_t *__restrict__ X, int M, const int32_t *__restrict__ idx,
                     const int32_t *__restrict__ count, int coff, const void *__restrict__ Wany,
                     const uint16_t *__restrict__ scales, const uint8_t *__restrict__ zeros, int N,
                     int K, int g_size, void *__restrict__ Y) {
    const int rows = count ? min(*count - coff, M) : M;
    const int lane = threadIdx.x & 31;
    const int n = (int)(((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    if (n >= N) return;
    const int G = MODE == 0 ? 1 : K / g_size;
    for (int slot = 0; slot < rows; ++slot) {
        const int row = idx ? idx[slot] : slot;
        float acc = 0.f;
        for (int k0 = lane * 8; k0 < K; k0 += 256) {
            float w[8];
            if (MODE == 0) {
                const uint16_t *wp = reinterpret_cast<const uint16_t *>(Wany) + (size_t)n * K + k0;
#pragma unroll
                for (int j = 0; j < 8; ++j) w[j] = __uint_as_float((uint32_t)wp[j] << 16);
            } else {
                const float s = __uint_as_float((uint32_t)scales[(size_t)n * G + k0 / g_size] << 16);
                const float z = (float)zeros[(size_t)n * G + k0 / g_size];
                const uint32_t *qp = reinterpret_cast<const uint32_t *>(Wany);
                if (MODE == 3) {
                    const uint32_t *u = qp + (size_t)n * (K / 32 * 3) + (size_t)(k0 / 32) * 3;
                    const uint32_t u0 = u[0], u1 = u[1], u2 = u[2];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int i = k0 % 32 + j;  // code i < 30: word i / 10, five codes per half-word; codes 30, 31: bits 15, 31
                        uint32_t q;
                        if (i < 30) {
                            const int jj = i % 10;
                            q = ((i < 10 ? u0 : (i < 20 ? u1 : u2)) >> (jj < 5 ? 3 * jj : 16 + 3 * (jj - 5))) & 7u;
                        } else {
                            const int bit = i == 30 ? 15 : 31;
                            q = ((u0 >> bit) & 1u) | (((u1 >> bit) & 1u) << 1) | (((u2 >> bit) & 1u) << 2);
                        }
                        w[j] = s * ((float)q - z);
                    }
                } else if (MODE == 4) {
                    const uint32_t u = qp[(size_t)n * (K / 8) + k0 / 8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) w[j] = s * ((float)((u >> (4 * j)) & 0xFu) - z);
                } else {
                    const uint32_t u0 = qp[(size_t)n * (K / 4) + k0 / 4], u1 = qp[(size_t)n * (K / 4) + k0 / 4 + 1];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        w[j] = s * ((float)((u0 >> (8 * j)) & 0xFFu) - z);
                        w[4 + j] = s * ((float)((u1 >> (8 * j)) & 0xFFu) - z);
                    }
                }
            }
            const uint16_t *xp = X + (size_t)row * K + k0;
#pragma unroll
            for (int j = 0; j < 8; ++j) acc = fmaf(__uint_as_float((uint32_t)xp[j] << 16), w[j], acc);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) {
            if (OUT_F32)
                reinterpret_cast<float *>(Y)[(size_t)row * N + n] = acc;
            else
                reinterpret_cast<__nv_bfloat16 *>(Y)[(size_t)row * N + n] = __float2bfloat16_rn(acc);
        }
    }
}

}  // namespace

dmr_status_t launch_simple_lowbit(const uint16_t *X, int M, RowSel sel, const uint32_t *qweight,
                                  const uint16_t *scales, const uint8_t *zeros, int N, int K, int bits,
                                  int g, void *Y, dmr_out_t out, cudaStream_t st) {
    const int grid = (N + 7) / 8;
    if (bits == 3) {
        if (out == DMR_OUT_F32)
            simple_linear_kernel<3, true><<<grid, 256, 0, st>>>(X, M, sel.idx, sel.count, sel.offset, qweight, scales, zeros, N, K, g, Y);
        else
            simple_linear_kernel<3, false><<<grid, 256, 0, st>>>(X, M, sel.idx, sel.count, sel.offset, qweight, scales, zeros, N, K, g, Y);
    } else if (bits == 4) {
        if (out == DMR_OUT_F32)
            simple_linear_kernel<4, true><<<grid, 256, 0, st>>>(X, M, sel.idx, sel.count, sel.offset, qweight, scales, zeros, N, K, g, Y);
        else
            simple_linear_kernel<4, false><<<grid, 256, 0, st>>>(X, M, sel.idx, sel.count, sel.offset, qweight, scales, zeros, N, K, g, Y);
    } else {
        if (out == DMR_OUT_F32)
            simple_linear_kernel<8, true><<<grid, 256, 0, st>>>(X, M, sel.idx, sel.count, sel.offset, qweight, scales, zeros, N, K, g, Y);
        else
            simple_linear_kernel<8, false><<<grid, 256, 0, st>>>(X, M, sel.idx, sel.count, sel.offset, qweight, scales, zeros, N, K, g, Y);
    }
    return check_launch();
}

dmr_status_t launch_simple_dense(const uint16_t *X, int M, RowSel sel, const uint16_t *W, int N, int K,
                                 void *Y, dmr_out_t out, cudaStream_t st) {
    const int grid = (N + 7) / 8;
    if (out == DMR_OUT_F32)
        simple_linear_kernel<0, true><<<grid, 256, 0, st>>>(X, M, sel.idx, sel.count, sel.offset, W, nullptr, nullptr, N, K, K, Y);
    else
        simple_linear_kernel<0, false><<<grid, 256, 0, st>>>(X, M, sel.idx, sel.count, sel.offset, W, nullptr, nullptr, N, K, K, Y);
    return check_launch();
}

}  // namespace dmr
