// Step-wise KL divergence between the action distributions of the high- and the low-precision
// model: KL_t = mean over the action tokens i of step t of KL(pi_high(x_i) || pi_low(x_i)), the
// quantity the KL-ST router is trained to predict (Sec. "KL-ST Stage"; App. on search and click
// steps, definition of the per-step action-block KL).
//
// Per token, with a = high-precision logits, b = low-precision logits, p = softmax(a):
//   KL = sum_v p_v (a_v - b_v) - lse(a) + lse(b),
// formed in ONE pass over the two logit rows (2 x V elements, read once: the kernel is bound by
// memory bandwidth) with running maxima, in fp32:
//   m_a, S0 = sum e^(a - m_a), S1 = sum e^(a - m_a) (a - b);   m_b, S2 = sum e^(b - m_b)
//   KL = S1 / S0 + ((m_b - m_a) + (log S2 - log S0)).
// A vocabulary entry with p_v = 0 (a_v = -inf) contributes nothing.  One CTA per token; threads
// keep private running sums, which are combined in a fixed order (lanes, then warps), so the result
// does not depend on the grid.  A second, tiny kernel averages the tokens of each step in order.
#include <cuda_bf16.h>

#include "common.cuh"

namespace dmr {

namespace {

constexpr int kKlThreads = 512;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kLogitFloor = -1.0e30f;  // -inf logits are raised to this: no inf - inf anywhere, e^(x - m) is still 0

struct KlState {
    float ma, s0, s1;  // maximum of a (in log2 units: a * log2 e), sum e^(a - ma), sum e^(a - ma) (a - b)
    float mb, s2;      // the same maximum and sum for b
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Adds elements (a_i, b_i), i < n, to the running sums; the maxima are raised once per call.
template <int n>
__device__ __forceinline__ void kl_update(KlState &st, const float (&a)[n], const float (&b)[n]) {
    float va = kLogitFloor, vb = kLogitFloor;
#pragma unroll
    for (int i = 0; i < n; ++i) {
        va = fmaxf(va, a[i]);
        vb = fmaxf(vb, b[i]);
    }
    va *= kLog2e;
    vb *= kLog2e;
    if (va > st.ma) {
        const float r = ex2(st.ma - va);  // 0 when the old maximum was -inf
        st.s0 *= r;
        st.s1 *= r;
        st.ma = va;
    }
    if (vb > st.mb) {
        st.s2 *= ex2(st.mb - vb);
        st.mb = vb;
    }
#pragma unroll
    for (int i = 0; i < n; ++i) {
        const float ai = fmaxf(a[i], kLogitFloor), bi = fmaxf(b[i], kLogitFloor);
        const float w = ex2(fmaf(ai, kLog2e, -st.ma));
        st.s0 += w;
        if (w > 0.f) st.s1 = fmaf(w, ai - bi, st.s1);  // p_v = 0 contributes nothing, whatever b_v is
        st.s2 += ex2(fmaf(bi, kLog2e, -st.mb));
    }
}

// st = st (+) o, the sums brought to the common maxima; `st` is the earlier part of the row.
__device__ __forceinline__ void kl_merge(KlState &st, const KlState &o) {
    const float ma = fmaxf(st.ma, o.ma), mb = fmaxf(st.mb, o.mb);
    const float r1 = st.ma == ma ? 1.f : ex2(st.ma - ma), r2 = o.ma == ma ? 1.f : ex2(o.ma - ma);
    st.s0 = st.s0 * r1 + o.s0 * r2;
    st.s1 = st.s1 * r1 + o.s1 * r2;
    st.ma = ma;
    const float q1 = st.mb == mb ? 1.f : ex2(st.mb - mb), q2 = o.mb == mb ? 1.f : ex2(o.mb - mb);
    st.s2 = st.s2 * q1 + o.s2 * q2;
    st.mb = mb;
}

__device__ __forceinline__ void unpack_bf16x8(const uint4 &q, float (&f)[8]) {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

// F32 = logits are fp32 (else bf16).  VEC = rows start on 16-byte boundaries (V a multiple of 8 or 4).
template <bool F32, bool VEC>
__global__ void __launch_bounds__(kKlThreads)
kl_token_kernel(const void *__restrict__ high, const void *__restrict__ low, int T, int V, float *__restrict__ kl_token) {
    __shared__ KlState warp_state[kKlThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int tok = blockIdx.x; tok < T; tok += gridDim.x) {
        KlState st = {-INFINITY, 0.f, 0.f, -INFINITY, 0.f};
        if (F32) {
            const float *a = reinterpret_cast<const float *>(high) + (size_t)tok * V;
            const float *b = reinterpret_cast<const float *>(low) + (size_t)tok * V;
            if (VEC) {
                const int nv = V / 4;
                for (int v = threadIdx.x; v < nv; v += kKlThreads) {
                    const float4 qa = __ldcs(reinterpret_cast<const float4 *>(a) + v);
                    const float4 qb = __ldcs(reinterpret_cast<const float4 *>(b) + v);
                    const float fa[4] = {qa.x, qa.y, qa.z, qa.w}, fb[4] = {qb.x, qb.y, qb.z, qb.w};
                    kl_update<4>(st, fa, fb);
                }
            } else {
                for (int v = threadIdx.x; v < V; v += kKlThreads) {
                    const float fa[1] = {a[v]}, fb[1] = {b[v]};
                    kl_update<1>(st, fa, fb);
                }
            }
        } else {
            const uint16_t *a = reinterpret_cast<const uint16_t *>(high) + (size_t)tok * V;
            const uint16_t *b = reinterpret_cast<const uint16_t *>(low) + (size_t)tok * V;
            if (VEC) {
                const int nv = V / 8;
                int v = threadIdx.x;
                // two 16-byte loads of each row in flight per thread
                for (; v + kKlThreads < nv; v += 2 * kKlThreads) {
                    const uint4 qa0 = __ldcs(reinterpret_cast<const uint4 *>(a) + v);
                    const uint4 qb0 = __ldcs(reinterpret_cast<const uint4 *>(b) + v);
                    const uint4 qa1 = __ldcs(reinterpret_cast<const uint4 *>(a) + v + kKlThreads);
                    const uint4 qb1 = __ldcs(reinterpret_cast<const uint4 *>(b) + v + kKlThreads);
                    float fa[8], fb[8];
                    unpack_bf16x8(qa0, fa);
                    unpack_bf16x8(qb0, fb);
                    kl_update<8>(st, fa, fb);
                    unpack_bf16x8(qa1, fa);
                    unpack_bf16x8(qb1, fb);
                    kl_update<8>(st, fa, fb);
                }
                if (v < nv) {
                    float fa[8], fb[8];
                    unpack_bf16x8(__ldcs(reinterpret_cast<const uint4 *>(a) + v), fa);
                    unpack_bf16x8(__ldcs(reinterpret_cast<const uint4 *>(b) + v), fb);
                    kl_update<8>(st, fa, fb);
                }
            } else {
                for (int v = threadIdx.x; v < V; v += kKlThreads) {
                    const float fa[1] = {__uint_as_float((uint32_t)a[v] << 16)}, fb[1] = {__uint_as_float((uint32_t)b[v] << 16)};
                    kl_update<1>(st, fa, fb);
                }
            }
        }
        // lanes (butterfly: every lane ends with the same sums), then warps in order
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            KlState other;
            other.ma = __shfl_xor_sync(0xFFFFFFFFu, st.ma, o);
            other.s0 = __shfl_xor_sync(0xFFFFFFFFu, st.s0, o);
            other.s1 = __shfl_xor_sync(0xFFFFFFFFu, st.s1, o);
            other.mb = __shfl_xor_sync(0xFFFFFFFFu, st.mb, o);
            other.s2 = __shfl_xor_sync(0xFFFFFFFFu, st.s2, o);
            // the lower lane's part comes first in both partners, so both compute the same value
            if (lane & o) {
                KlState first = other;
                kl_merge(first, st);
                st = first;
            } else {
                kl_merge(st, other);
            }
        }
        __syncthreads();  // warp_state of the previous token has been read
        if (lane == 0) warp_state[warp] = st;
        __syncthreads();
        if (threadIdx.x == 0) {
            KlState tot = warp_state[0];
            for (int w = 1; w < kKlThreads / 32; ++w) kl_merge(tot, warp_state[w]);
            // lse(b) - lse(a), differences first (exactly 0 for equal rows), from log2 to natural-log units
            const float dlse = ((tot.mb - tot.ma) + (log2f(tot.s2) - log2f(tot.s0))) * kLn2;
            kl_token[tok] = tot.s1 / tot.s0 + dlse;
        }
    }
}

// kl_step[s] = mean of kl_token over [offsets[s], offsets[s + 1]), added in token order; 0 for an empty step.
__global__ void __launch_bounds__(128)
kl_step_kernel(const float *__restrict__ kl_token, const int32_t *__restrict__ offsets, int S, int T, float *__restrict__ kl_step) {
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= S) return;
    int beg = offsets[s], end = offsets[s + 1];
    beg = beg < 0 ? 0 : beg;
    end = end > T ? T : end;
    float sum = 0.f;
    for (int i = beg; i < end; ++i) sum += kl_token[i];
    kl_step[s] = end > beg ? sum / (float)(end - beg) : 0.f;
}

}  // namespace

dmr_status_t launch_stepwise_kl(const void *high, const void *low, bool f32, int T, int V, const int32_t *offsets, int S,
                                float *kl_token, float *kl_step, cudaStream_t st) {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) sms = n;
    }
    const int blocks = T < sms * 8 ? T : sms * 8;
    const bool vec = V % (f32 ? 4 : 8) == 0;
    if (T == 0) {
        // no tokens: only the (zero) step means are written
    } else if (f32) {
        if (vec) kl_token_kernel<true, true><<<blocks, kKlThreads, 0, st>>>(high, low, T, V, kl_token);
        else kl_token_kernel<true, false><<<blocks, kKlThreads, 0, st>>>(high, low, T, V, kl_token);
    } else {
        if (vec) kl_token_kernel<false, true><<<blocks, kKlThreads, 0, st>>>(high, low, T, V, kl_token);
        else kl_token_kernel<false, false><<<blocks, kKlThreads, 0, st>>>(high, low, T, V, kl_token);
    }
    dmr_status_t r = check_launch();
    if (r != DMR_OK || S == 0) return r;
    kl_step_kernel<<<(S + 127) / 128, 128, 0, st>>>(kl_token, offsets, S, T, kl_step);
    return check_launch();
}

}  // namespace dmr
