// Weight packer: bf16 weights -> packed unsigned codes (3, 4 or 8 bits) + per-group bf16 scale and u8 zero point,
// and the matching dequantizer (test utility).
//
// The low-precision model is weight-only quantization of the decoder Linear layers with 16-bit
// activations (Sec. 5 "Experimental Models and Precision", App. "Quantization Detail").  The rule
// implemented is asymmetric min/max round-to-nearest, evaluated in binary64 so that the integer
// decisions (zero point, codes) are taken in one fixed precision:
//   lo = min(0, min w), hi = max(0, max w), s = bf16_rne((hi - lo) / qmax), zero = rint(-lo / s),
//   code = clamp(rint(w / s) + zero, 0, qmax).
#include "common.cuh"

namespace dmr {

namespace {

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

// Nearest bf16 (ties to even) of a positive finite double, never below the smallest normal.
__device__ __forceinline__ uint32_t scale_to_bf16(double x) {
    unsigned long long u = (unsigned long long)__double_as_longlong(x);
    int e = (int)((u >> 52) & 0x7FFull) - 1023 + 127;   // bf16 biased exponent
    if (e <= 0) return 0x0080u;                          // below 2^-126: use 2^-126
    unsigned long long man = u & ((1ull << 52) - 1);
    uint32_t m7 = (uint32_t)(man >> 45);
    unsigned long long rem = man & ((1ull << 45) - 1);
    uint32_t r = ((uint32_t)e << 7) | m7;
    const unsigned long long half = 1ull << 44;
    if (rem > half || (rem == half && (m7 & 1u))) ++r;   // a carry moves into the exponent
    return r;
}

// One warp per (row, group).  Lanes take 8 consecutive weights at a time (one 16-byte load).
template <int BITS>
__global__ void __launch_bounds__(256) quantize_kernel(const uint16_t *__restrict__ W, int N, int K,
                                                       int g, uint32_t *__restrict__ qweight,
                                                       uint16_t *__restrict__ scales,
                                                       uint8_t *__restrict__ zeros,
                                                       int32_t *__restrict__ dev_status) {
    const int lane = threadIdx.x & 31;
    const int G = K / g;
    const long long total = (long long)N * G;
    const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    const double qmax = (double)((1 << BITS) - 1);
    const int chunks = g / 8;

    for (long long item = warp0; item < total; item += nwarps) {
        const int n = (int)(item / G);
        const int j = (int)(item % G);
        const uint16_t *wg = W + (size_t)n * K + (size_t)j * g;

        // pass 1: range of the group (bf16 -> float is exact, so float min/max is exact)
        float lo = 0.f, hi = 0.f;
        bool bad = false;
        for (int c = lane; c < chunks; c += 32) {
            uint4 v = *reinterpret_cast<const uint4 *>(wg + c * 8);
            uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t b0 = w[i] & 0xFFFFu, b1 = w[i] >> 16;
                bad |= ((b0 & 0x7F80u) == 0x7F80u) | ((b1 & 0x7F80u) == 0x7F80u);
                float f0 = bf16_bits_to_float(b0), f1 = bf16_bits_to_float(b1);
                lo = fminf(lo, fminf(f0, f1));
                hi = fmaxf(hi, fmaxf(f0, f1));
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            lo = fminf(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, o));
            hi = fmaxf(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, o));
        }
        bad = __any_sync(0xFFFFFFFFu, bad);
        if (bad) {
            if (lane == 0 && dev_status) atomicExch(dev_status, (int)DMR_ERR_NONFINITE);
            continue;
        }

        // scale and zero point, binary64
        const double dlo = (double)lo, dhi = (double)hi;
        uint32_t sb = (dhi == dlo) ? 0x3F80u : scale_to_bf16(__ddiv_rn(__dsub_rn(dhi, dlo), qmax));
        if (sb < 0x0080u) sb = 0x0080u;
        const double s = (double)bf16_bits_to_float(sb);
        double z = rint(__ddiv_rn(-dlo, s));
        z = fmin(fmax(z, 0.0), qmax);
        if (lane == 0) {
            scales[(size_t)n * G + j] = (uint16_t)sb;
            zeros[(size_t)n * G + j] = (uint8_t)z;
        }

        // pass 2: codes, 8 per lane per step, packed little-endian in k (every lane takes every step of the loop:
        // the 3-bit words are put together from four neighbouring lanes)
        for (int c0 = 0; c0 < chunks; c0 += 32) {
            const int c = c0 + lane;
            const bool active = c < chunks;
            uint32_t q[8];
            if (active) {
                uint4 v = *reinterpret_cast<const uint4 *>(wg + c * 8);
                uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        double x = (double)bf16_bits_to_float(h ? (w[i] >> 16) : (w[i] & 0xFFFFu));
                        double c2 = __dadd_rn(rint(__ddiv_rn(x, s)), z);
                        c2 = fmin(fmax(c2, 0.0), qmax);
                        q[2 * i + h] = (uint32_t)c2;
                    }
                }
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) q[i] = 0;
            }
            const size_t k0 = (size_t)j * g + (size_t)c * 8;
            if (BITS == 4) {
                uint32_t word = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) word |= q[i] << (4 * i);
                if (active) qweight[(size_t)n * (K / 8) + k0 / 8] = word;
            } else if (BITS == 8) {
                uint32_t w0 = q[0] | (q[1] << 8) | (q[2] << 16) | (q[3] << 24);
                uint32_t w1 = q[4] | (q[5] << 8) | (q[6] << 16) | (q[7] << 24);
                if (active) *reinterpret_cast<uint2 *>(qweight + (size_t)n * (K / 4) + k0 / 4) = make_uint2(w0, w1);
            } else {
                // 32 codes in three words: code i < 30 in word i / 10, five codes in each half-word; the bits of codes
                // 30 and 31 in bit 15 and bit 31 of the three words.  Four lanes hold one block of 32 codes.
                uint32_t p[3] = {0u, 0u, 0u};
                const int pos = (c & 3) * 8;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int i = pos + e;
                    if (i < 30) {
                        const int jj = i % 10;
                        const uint32_t v = q[e] << (jj < 5 ? 3 * jj : 16 + 3 * (jj - 5));
                        const int word = i / 10;
                        p[0] |= word == 0 ? v : 0u;
                        p[1] |= word == 1 ? v : 0u;
                        p[2] |= word == 2 ? v : 0u;
                    } else {
                        const int bit = i == 30 ? 15 : 31;
#pragma unroll
                        for (int b = 0; b < 3; ++b) p[b] |= ((q[e] >> b) & 1u) << bit;
                    }
                }
#pragma unroll
                for (int b = 0; b < 3; ++b) {
                    p[b] |= __shfl_xor_sync(0xFFFFFFFFu, p[b], 1);
                    p[b] |= __shfl_xor_sync(0xFFFFFFFFu, p[b], 2);
                }
                if (active && (c & 3) == 0) {
                    uint32_t *dst = qweight + (size_t)n * (K / 32 * 3) + k0 / 32 * 3;
                    dst[0] = p[0];
                    dst[1] = p[1];
                    dst[2] = p[2];
                }
            }
        }
    }
}

// One thread per 8 consecutive weights of a row.
template <int BITS, bool OUT_F32>
__global__ void __launch_bounds__(256) dequantize_kernel(const uint32_t *__restrict__ qweight,
                                                         const uint16_t *__restrict__ scales,
                                                         const uint8_t *__restrict__ zeros, int N,
                                                         int K, int g, void *__restrict__ out) {
    const long long total = (long long)N * (K / 8);
    const int G = K / g;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int n = (int)(i / (K / 8));
        const int k0 = (int)(i % (K / 8)) * 8;
        const float s = bf16_bits_to_float(scales[(size_t)n * G + k0 / g]);
        const float z = (float)zeros[(size_t)n * G + k0 / g];
        uint32_t q[8];
        if (BITS == 3) {
            const uint32_t *w = qweight + (size_t)n * (K / 32 * 3) + (size_t)(k0 / 32) * 3;
            const uint32_t w0 = w[0], w1 = w[1], w2 = w[2];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int i = k0 % 32 + j;
                if (i < 30) {
                    const int jj = i % 10;
                    const uint32_t word = i < 10 ? w0 : (i < 20 ? w1 : w2);
                    q[j] = (word >> (jj < 5 ? 3 * jj : 16 + 3 * (jj - 5))) & 7u;
                } else {
                    const int bit = i == 30 ? 15 : 31;
                    q[j] = ((w0 >> bit) & 1u) | (((w1 >> bit) & 1u) << 1) | (((w2 >> bit) & 1u) << 2);
                }
            }
        } else if (BITS == 4) {
            uint32_t w = qweight[(size_t)n * (K / 8) + k0 / 8];
#pragma unroll
            for (int j = 0; j < 8; ++j) q[j] = (w >> (4 * j)) & 0xFu;
        } else {
            uint2 w = *reinterpret_cast<const uint2 *>(qweight + (size_t)n * (K / 4) + k0 / 4);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                q[j] = (w.x >> (8 * j)) & 0xFFu;
                q[4 + j] = (w.y >> (8 * j)) & 0xFFu;
            }
        }
        float v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = __fmul_rn(s, (float)q[j] - z);  // exact: 8 x 9 significant bits
        if (OUT_F32) {
            float4 *o = reinterpret_cast<float4 *>((float *)out + (size_t)n * K + k0);
            o[0] = make_float4(v[0], v[1], v[2], v[3]);
            o[1] = make_float4(v[4], v[5], v[6], v[7]);
        } else {
            uint32_t p[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                // round to nearest even bf16 by integer arithmetic on the fp32 pattern (values are finite)
                uint32_t a = __float_as_uint(v[2 * j]), b = __float_as_uint(v[2 * j + 1]);
                a = (a + 0x7FFFu + ((a >> 16) & 1u)) >> 16;
                b = (b + 0x7FFFu + ((b >> 16) & 1u)) >> 16;
                p[j] = a | (b << 16);
            }
            *reinterpret_cast<uint4 *>((uint16_t *)out + (size_t)n * K + k0) = make_uint4(p[0], p[1], p[2], p[3]);
        }
    }
}

}  // namespace

dmr_status_t launch_quantize(const uint16_t *W, int N, int K, int bits, int g, uint32_t *qweight,
                             uint16_t *scales, uint8_t *zeros, int32_t *dev_status, cudaStream_t st) {
    const long long items = (long long)N * (K / g);
    const int warps_per_block = 8;
    long long blocks = (items + warps_per_block - 1) / warps_per_block;
    if (blocks > 148 * 32) blocks = 148 * 32;
    if (bits == 3)
        quantize_kernel<3><<<(int)blocks, 256, 0, st>>>(W, N, K, g, qweight, scales, zeros, dev_status);
    else if (bits == 4)
        quantize_kernel<4><<<(int)blocks, 256, 0, st>>>(W, N, K, g, qweight, scales, zeros, dev_status);
    else
        quantize_kernel<8><<<(int)blocks, 256, 0, st>>>(W, N, K, g, qweight, scales, zeros, dev_status);
    return check_launch();
}

dmr_status_t launch_dequantize(const uint32_t *qweight, const uint16_t *scales, const uint8_t *zeros,
                               int N, int K, int bits, int g, void *W_out, dmr_out_t out, cudaStream_t st) {
    const long long total = (long long)N * (K / 8);
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 64) blocks = 148 * 64;
    if (bits == 3) {
        if (out == DMR_OUT_F32)
            dequantize_kernel<3, true><<<(int)blocks, 256, 0, st>>>(qweight, scales, zeros, N, K, g, W_out);
        else
            dequantize_kernel<3, false><<<(int)blocks, 256, 0, st>>>(qweight, scales, zeros, N, K, g, W_out);
    } else if (bits == 4) {
        if (out == DMR_OUT_F32)
            dequantize_kernel<4, true><<<(int)blocks, 256, 0, st>>>(qweight, scales, zeros, N, K, g, W_out);
        else
            dequantize_kernel<4, false><<<(int)blocks, 256, 0, st>>>(qweight, scales, zeros, N, K, g, W_out);
    } else {
        if (out == DMR_OUT_F32)
            dequantize_kernel<8, true><<<(int)blocks, 256, 0, st>>>(qweight, scales, zeros, N, K, g, W_out);
        else
            dequantize_kernel<8, false><<<(int)blocks, 256, 0, st>>>(qweight, scales, zeros, N, K, g, W_out);
    }
    return check_launch();
}

}  // namespace dmr
