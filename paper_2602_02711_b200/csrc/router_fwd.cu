// Forward pass of the step-level router (Sec. 4.1 "Router Architecture"):
//     H_t = TransformerEnc_theta(X_t + P_t, m_t),    pi_theta(r_t | s_t) = Softmax(W h_t*),
// X_t = [z_task, z_1, ..., z_t] the embeddings of the task and of the steps so far, P_t learned positional
// embeddings, m_t the valid-step mask (here: a length per sequence, valid steps first), h_t* the encoder's output at
// the last valid step.  The probabilities go to dmr_router_calibrate / dmr_router_mask and from there to
// dmr_routed_linear without leaving the device.
//
// The paper fixes neither width, heads, feed-forward size, normalisation placement nor activation.  Reading taken: the
// encoder layer of the original Transformer - x <- LN(x + MHA(x)), x <- LN(x + W2 relu(W1 x + b1) + b2), scaled
// dot-product attention in which padded steps are never keys (attention among the valid steps is not causal: the
// sequence already ends at the step being decided), LN over the feature axis with eps = 1e-5, no dropout.
//
// Arithmetic: fp32 throughout (CUDA cores; fused multiply-adds), so that the probabilities agree with a binary64
// evaluation to about 1e-6 and the comparison against a threshold is stable.  The model is small (14 M parameters at
// d = 384 and 8 layers) and runs once per agent step, next to a language-model call of tens of milliseconds.
// Kernels: positions added; per layer a linear (QKV; tiled, or one feature per warp when there are at most 32 tokens), one CTA per (sequence, head) for the attention, a linear
// with the residual added, a layer norm, two linears (ReLU; residual), a layer norm; then pooling, head and softmax.
#include "sm100.cuh"

namespace dmr {

namespace {

constexpr float kLnEps = 1e-5f;

// Lengths come from the caller's device memory and are not checked on the host: keep every index in range.
__device__ __forceinline__ int valid_len(int n, int L) { return n < 1 ? 1 : (n > L ? L : n); }

// H[b][l][:] = Z[b][l][:] + P[l][:] for the valid steps, zero behind them.
__global__ void __launch_bounds__(256) router_embed_kernel(const float *__restrict__ Z, const float *__restrict__ pos,
                                                           const int32_t *__restrict__ lengths, int B, int L, int d,
                                                           float *__restrict__ H) {
    const long long total = (long long)B * L * (d / 4);
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int c4 = (int)(i % (d / 4));
        const int l = (int)((i / (d / 4)) % L);
        const int b = (int)(i / ((long long)(d / 4) * L));
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (l < valid_len(lengths[b], L)) {
            const float4 z = reinterpret_cast<const float4 *>(Z)[i];
            const float4 p = reinterpret_cast<const float4 *>(pos)[(size_t)l * (d / 4) + c4];
            v = make_float4(z.x + p.x, z.y + p.y, z.z + p.z, z.w + p.w);
        }
        reinterpret_cast<float4 *>(H)[i] = v;
    }
}

// Y[T][N] = act(X[T][K] W[N][K]^T + bias) (+ R[T][N]).  64 x 64 output tile per CTA, 16-wide k steps, 4 x 4 outputs per
// thread.  K is a multiple of 16; T and N are arbitrary.
constexpr int LBM = 64, LBN = 64, LBK = 16;
template <bool RELU, bool RESID>
__global__ void __launch_bounds__(256) router_linear_kernel(const float *__restrict__ X, const float *__restrict__ W,
                                                            const float *__restrict__ bias, const float *__restrict__ R,
                                                            int T, int N, int K, float *__restrict__ Y) {
    __shared__ float xs[LBK][LBM + 4];
    __shared__ float ws[LBK][LBN + 4];
    const int t0 = blockIdx.y * LBM, n0 = blockIdx.x * LBN;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;  // outputs (t0 + 4 ty + i, n0 + 4 tx + j)
    const int lr = threadIdx.x >> 2, lc = (threadIdx.x & 3) * 4;  // this thread's 4 consecutive k of row lr of each tile
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int k0 = 0; k0 < K; k0 += LBK) {
        float4 xv = make_float4(0.f, 0.f, 0.f, 0.f), wv = xv;
        if (t0 + lr < T) xv = *reinterpret_cast<const float4 *>(X + (size_t)(t0 + lr) * K + k0 + lc);
        if (n0 + lr < N) wv = *reinterpret_cast<const float4 *>(W + (size_t)(n0 + lr) * K + k0 + lc);
        xs[lc + 0][lr] = xv.x;
        xs[lc + 1][lr] = xv.y;
        xs[lc + 2][lr] = xv.z;
        xs[lc + 3][lr] = xv.w;
        ws[lc + 0][lr] = wv.x;
        ws[lc + 1][lr] = wv.y;
        ws[lc + 2][lr] = wv.z;
        ws[lc + 3][lr] = wv.w;
        __syncthreads();
#pragma unroll
        for (int k = 0; k < LBK; ++k) {
            const float4 a = *reinterpret_cast<const float4 *>(&xs[k][4 * ty]);
            const float4 b = *reinterpret_cast<const float4 *>(&ws[k][4 * tx]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int t = t0 + 4 * ty + i;
        if (t >= T) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + 4 * tx + j;
            if (n >= N) continue;
            float v = acc[i][j] + bias[n];
            if (RELU) v = fmaxf(v, 0.f);
            if (RESID) v += R[(size_t)t * N + n];
            Y[(size_t)t * N + n] = v;
        }
    }
}

// The same linear for at most 32 tokens (one agent deciding one step): a 64 x 64 tile per CTA would leave most SMs idle,
// so a CTA takes two output features and all tokens, four warps per feature each with a quarter of the k range - the
// weight row is read once, 16 bytes per lane, the activations come through the L1 - and the sums are reduced across
// the warp and then across the four warps (in a fixed order) at the end.
constexpr int kSmallT = 32;
template <bool RELU, bool RESID>
__global__ void __launch_bounds__(256) router_linear_small_kernel(const float *__restrict__ X, const float *__restrict__ W,
                                                                  const float *__restrict__ bias, const float *__restrict__ R,
                                                                  int T, int N, int K, float *__restrict__ Y) {
    __shared__ float part[2][4][kSmallT];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int f = warp >> 2, ks = warp & 3;
    const int n = blockIdx.x * 2 + f;
    const int kq = K / 4;  // K is a multiple of 16
    float acc[kSmallT];
#pragma unroll
    for (int t = 0; t < kSmallT; ++t) acc[t] = 0.f;
    if (n < N) {
        for (int k = ks * kq + 4 * lane; k < (ks + 1) * kq; k += 128) {
            const float4 w = __ldg(reinterpret_cast<const float4 *>(W + (size_t)n * K + k));
#pragma unroll
            for (int t = 0; t < kSmallT; ++t) {
                if (t < T) {
                    const float4 x = __ldg(reinterpret_cast<const float4 *>(X + (size_t)t * K + k));
                    acc[t] = fmaf(w.x, x.x, fmaf(w.y, x.y, fmaf(w.z, x.z, fmaf(w.w, x.w, acc[t]))));
                }
            }
        }
    }
    float mine = 0.f;  // lane t keeps token t's sum
#pragma unroll
    for (int t = 0; t < kSmallT; ++t) {
        float v = acc[t];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        if (lane == t) mine = v;
    }
    part[f][ks][lane] = mine;
    __syncthreads();
    if (ks == 0 && n < N && lane < T) {
        float v = ((part[f][0][lane] + part[f][1][lane]) + part[f][2][lane]) + part[f][3][lane] + bias[n];
        if (RELU) v = fmaxf(v, 0.f);
        if (RESID) v += R[(size_t)lane * N + n];
        Y[(size_t)lane * N + n] = v;
    }
}

// One CTA per (sequence, head): softmax(Q K^T / sqrt(dh)) V over the valid steps.  QKV [T][3 d] (queries, keys, values),
// O [T][d].  Keys and values of the head sit in shared memory (rows padded by one float); a warp takes query rows
// warp, warp + 4, ...; every lane scores the keys lane, lane + 32, ... (L <= 128) and then sums its columns of V.
constexpr int kAttWarps = 4, kAttMaxL = 128;
__global__ void __launch_bounds__(kAttWarps * 32) router_attention_kernel(const float *__restrict__ QKV,
                                                                          const int32_t *__restrict__ lengths, int L, int d,
                                                                          int dh, float *__restrict__ O) {
    extern __shared__ float att_smem[];
    const int b = blockIdx.x, h = blockIdx.y;
    const int n = valid_len(lengths[b], L);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float *ks = att_smem;                       // [L][dh + 1]
    float *vs = ks + (size_t)L * (dh + 1);      // [L][dh + 1]
    float *ps = vs + (size_t)L * (dh + 1);      // [warps][L]: a query row's probabilities
    float *qs = ps + (size_t)kAttWarps * L;     // [warps][dh]
    const size_t row0 = (size_t)b * L;
    for (int i = threadIdx.x; i < n * dh; i += blockDim.x) {
        const int j = i / dh, c = i % dh;
        const float *src = QKV + (row0 + j) * (size_t)(3 * d) + h * dh + c;
        ks[j * (dh + 1) + c] = src[d];
        vs[j * (dh + 1) + c] = src[2 * d];
    }
    __syncthreads();
    const float scale = 1.0f / sqrtf((float)dh);
    // this CTA's share of the query rows (gridDim.z CTAs per sequence and head)
    const int rows_per = (L + gridDim.z - 1) / gridDim.z;
    const int l_lo = blockIdx.z * rows_per, l_hi = min(L, l_lo + rows_per);
    for (int l = l_lo + warp; l < l_hi; l += kAttWarps) {
        float *orow = O + (row0 + l) * (size_t)d + h * dh;
        if (l >= n) {  // a padded step: nothing reads its row; keep it finite
            for (int c = lane; c < dh; c += 32) orow[c] = 0.f;
            continue;
        }
        for (int c = lane; c < dh; c += 32) qs[warp * dh + c] = QKV[(row0 + l) * (size_t)(3 * d) + h * dh + c];
        __syncwarp();
        float s[kAttMaxL / 32];
        float mx = -INFINITY;
#pragma unroll
        for (int u = 0; u < kAttMaxL / 32; ++u) {
            const int j = lane + 32 * u;
            s[u] = -INFINITY;
            if (j < n) {
                float a = 0.f;
                for (int c = 0; c < dh; ++c) a = fmaf(qs[warp * dh + c], ks[j * (dh + 1) + c], a);
                s[u] = a * scale;
            }
            mx = fmaxf(mx, s[u]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
        float sum = 0.f;
#pragma unroll
        for (int u = 0; u < kAttMaxL / 32; ++u) {
            const int j = lane + 32 * u;
            const float e = j < n ? expf(s[u] - mx) : 0.f;
            if (j < L) ps[warp * L + j] = e;
            sum += e;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
        const float inv = 1.f / sum;
        __syncwarp();
        for (int c = lane; c < dh; c += 32) {
            float a = 0.f;
            for (int j = 0; j < n; ++j) a = fmaf(ps[warp * L + j], vs[j * (dh + 1) + c], a);
            orow[c] = a * inv;
        }
        __syncwarp();
    }
}

// One warp per token: H[t][:] = (x - mean) / sqrt(var + eps) * g + b over the d features of S[t][:] (d <= 1024).
__global__ void __launch_bounds__(256) router_layernorm_kernel(const float *__restrict__ S, const float *__restrict__ g,
                                                               const float *__restrict__ bta, int T, int d,
                                                               float *__restrict__ H) {
    const int t = (int)(((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    const int lane = threadIdx.x & 31;
    if (t >= T) return;
    float x[32];
    float sum = 0.f;
#pragma unroll
    for (int u = 0; u < 32; ++u) {
        const int c = lane + 32 * u;
        x[u] = c < d ? S[(size_t)t * d + c] : 0.f;
        sum += x[u];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
    const float mean = sum / (float)d;
    float sq = 0.f;
#pragma unroll
    for (int u = 0; u < 32; ++u) {
        const int c = lane + 32 * u;
        const float dv = c < d ? x[u] - mean : 0.f;
        sq = fmaf(dv, dv, sq);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xFFFFFFFFu, sq, o);
    const float rstd = 1.f / sqrtf(sq / (float)d + kLnEps);
#pragma unroll
    for (int u = 0; u < 32; ++u) {
        const int c = lane + 32 * u;
        if (c < d) H[(size_t)t * d + c] = (x[u] - mean) * rstd * g[c] + bta[c];
    }
}

// One CTA (one warp) per sequence: h* = H at the last valid step, logits = W h* + b, softmax over the classes (<= 32).
__global__ void __launch_bounds__(32) router_head_kernel(const float *__restrict__ H, const int32_t *__restrict__ lengths,
                                                         const float *__restrict__ wc, const float *__restrict__ bc, int L,
                                                         int d, int classes, int score_class, float *__restrict__ probs,
                                                         float *__restrict__ scores) {
    const int b = blockIdx.x, lane = threadIdx.x;
    const float *hstar = H + ((size_t)b * L + (valid_len(lengths[b], L) - 1)) * d;
    float mine = -INFINITY;  // lane c keeps the logit of class c
    for (int c = 0; c < classes; ++c) {
        float a = 0.f;
        for (int k = lane; k < d; k += 32) a = fmaf(wc[(size_t)c * d + k], hstar[k], a);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xFFFFFFFFu, a, o);
        if (lane == c) mine = a + bc[c];
    }
    float mx = mine;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
    const float e = lane < classes ? expf(mine - mx) : 0.f;
    float sum = e;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
    const float p = e / sum;
    if (lane < classes) probs[(size_t)b * classes + lane] = p;
    if (scores && lane == score_class) scores[b] = p;
}

template <bool RELU, bool RESID>
dmr_status_t launch_linear(const float *X, const float *W, const float *bias, const float *R, int T, int N, int K, float *Y,
                           cudaStream_t st) {
    if (T <= kSmallT) {
        router_linear_small_kernel<RELU, RESID><<<(N + 1) / 2, 256, 0, st>>>(X, W, bias, R, T, N, K, Y);
    } else {
        dim3 grid((unsigned)((N + LBN - 1) / LBN), (unsigned)((T + LBM - 1) / LBM), 1);
        router_linear_kernel<RELU, RESID><<<grid, 256, 0, st>>>(X, W, bias, R, T, N, K, Y);
    }
    return check_launch();
}

}  // namespace

size_t router_param_floats(const dmr_router_cfg_t &c) {
    const size_t d = (size_t)c.d, f = (size_t)c.ffn;
    const size_t per_layer = 3 * d * d + 3 * d + d * d + d + 2 * d + f * d + f + d * f + d + 2 * d;
    return (size_t)c.l_max * d + (size_t)c.layers * per_layer + (size_t)c.classes * d + (size_t)c.classes;
}

size_t router_workspace_bytes(const dmr_router_cfg_t &c, int B, int L) {
    const size_t T = (size_t)B * L;
    return round_up(T * (size_t)(6 * c.d + c.ffn) * sizeof(float), 256);
}

size_t router_attention_smem(int L, int dh) { return ((size_t)2 * L * (dh + 1) + (size_t)kAttWarps * L + (size_t)kAttWarps * dh) * sizeof(float); }

dmr_status_t launch_router_forward(const float *params, const dmr_router_cfg_t &c, const float *Z, const int32_t *lengths, int B,
                                   int L, float *probs, float *scores, int score_class, float *ws, cudaStream_t st) {
    const int d = c.d, f = c.ffn, T = B * L, dh = c.d / c.heads;
    float *H = ws;                        // [T][d]   the layer's input and output
    float *QKV = H + (size_t)T * d;       // [T][3 d]
    float *ATT = QKV + (size_t)T * 3 * d; // [T][d]   attention output
    float *SUM = ATT + (size_t)T * d;     // [T][d]   residual sums before a layer norm
    float *FF = SUM + (size_t)T * d;      // [T][f]
    const size_t att_smem = router_attention_smem(L, dh);
    if (!ensure_dynamic_smem(reinterpret_cast<const void *>(router_attention_kernel), att_smem)) return DMR_ERR_CUDA;
    dmr_status_t r;
    {
        const long long total = (long long)T * (d / 4);
        long long blocks = (total + 255) / 256;
        if (blocks > 148 * 16) blocks = 148 * 16;
        router_embed_kernel<<<(int)blocks, 256, 0, st>>>(Z, params, lengths, B, L, d, H);
        if ((r = check_launch()) != DMR_OK) return r;
    }
    const float *p = params + (size_t)c.l_max * d;
    const int ln_blocks = (T + 7) / 8;
    for (int layer = 0; layer < c.layers; ++layer) {
        const float *wqkv = p, *bqkv = wqkv + (size_t)3 * d * d, *wo = bqkv + 3 * d, *bo = wo + (size_t)d * d;
        const float *ln1_g = bo + d, *ln1_b = ln1_g + d, *w1 = ln1_b + d, *b1 = w1 + (size_t)f * d;
        const float *w2 = b1 + f, *b2 = w2 + (size_t)d * f, *ln2_g = b2 + d, *ln2_b = ln2_g + d;
        p = ln2_b + d;
        if ((r = launch_linear<false, false>(H, wqkv, bqkv, nullptr, T, 3 * d, d, QKV, st)) != DMR_OK) return r;
        // few sequences: split a sequence's query rows over several CTAs (each loads the head's keys and values again)
        int zsplit = (4 * 148) / (B * c.heads);
        zsplit = zsplit < 1 ? 1 : (zsplit > (L + kAttWarps - 1) / kAttWarps ? (L + kAttWarps - 1) / kAttWarps : zsplit);
        router_attention_kernel<<<dim3((unsigned)B, (unsigned)c.heads, (unsigned)zsplit), kAttWarps * 32, att_smem, st>>>(QKV, lengths, L, d, dh, ATT);
        if ((r = check_launch()) != DMR_OK) return r;
        if ((r = launch_linear<false, true>(ATT, wo, bo, H, T, d, d, SUM, st)) != DMR_OK) return r;
        router_layernorm_kernel<<<ln_blocks, 256, 0, st>>>(SUM, ln1_g, ln1_b, T, d, H);
        if ((r = check_launch()) != DMR_OK) return r;
        if ((r = launch_linear<true, false>(H, w1, b1, nullptr, T, f, d, FF, st)) != DMR_OK) return r;
        if ((r = launch_linear<false, true>(FF, w2, b2, H, T, d, f, SUM, st)) != DMR_OK) return r;
        router_layernorm_kernel<<<ln_blocks, 256, 0, st>>>(SUM, ln2_g, ln2_b, T, d, H);
        if ((r = check_launch()) != DMR_OK) return r;
    }
    router_head_kernel<<<B, 32, 0, st>>>(H, lengths, p, p + (size_t)c.classes * d, L, d, c.classes, score_class, probs, scores);
    return check_launch();
}

}  // namespace dmr
