// Shared declarations of the libdmr CUDA sources (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "dmr.h"

namespace dmr {

// ---- host-side bookkeeping -------------------------------------------------------------
extern std::atomic<int> g_last_cuda_error;           // last failing cudaError_t (0 if none)
extern std::atomic<unsigned long long> g_launches;   // kernels launched by this library in this process

inline dmr_status_t check_launch() {
    ++g_launches;
    cudaError_t e = cudaPeekAtLastError();
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        (void)cudaGetLastError();
        return DMR_ERR_CUDA;
    }
    return DMR_OK;
}

inline bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }

inline int group_of(int K, dmr_qformat_t f) { return f.group_size == 0 ? K : f.group_size; }

// A format is usable when: bits in {3,4,8}; K, g multiples of 32; g divides K.
inline bool format_ok(int K, dmr_qformat_t f) {
    if (f.bits != 3 && f.bits != 4 && f.bits != 8) return false;
    if (K <= 0 || K % 32 != 0) return false;
    int g = group_of(K, f);
    if (g <= 0 || g % 32 != 0 || K % g != 0) return false;
    return true;
}

// Row lists for routed calls: `idx` lists the rows of X/Y to process and `count` (device) says
// how many entries are valid.  Both null for a plain call over rows 0..M-1.
struct RowSel {
    const int32_t *idx;    // already advanced to the first slot of this launch
    const int32_t *count;  // total number of valid slots in the list
    int32_t offset;        // list position of this launch's first slot (subtracted from *count)
};

// ---- workspace layout --------------------------------------------------------------------
// [0, 256)            status word (int32) + padding
// [256, ...)          routed: counts[2] (+pad to 256), idx_high[Mpad], idx_low[Mpad]
// then                compacted activations / split-K partial sums, op dependent
constexpr size_t kWsStatusBytes = 256;

inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- kernel launchers (defined in the .cu files) ------------------------------------------
dmr_status_t launch_quantize(const uint16_t *W, int N, int K, int bits, int g, uint32_t *qweight,
                             uint16_t *scales, uint8_t *zeros, int32_t *dev_status,
                             cudaStream_t st);
dmr_status_t launch_dequantize(const uint32_t *qweight, const uint16_t *scales, const uint8_t *zeros,
                               int N, int K, int bits, int g, void *W_out, dmr_out_t out,
                               cudaStream_t st);

// Streaming decode kernel (M <= 32 per launch): persistent, one or two CTAs per SM, weights read once.  `bits` is 4 or 8
// for packed codes and 16 for bf16 weights.  `scratch` holds stream_scratch_bytes(N) bytes that are
// zero before the first use (the kernel leaves its counters zeroed again).
constexpr int kMaxStreamCtas = 512;
// Feature-group counters sit one per 128-byte line: counts into different groups then never queue up
// behind each other in the L2.
constexpr int kCounterStride = 32;  // int32 words between counters
// Scratch layout: per-CTA partial sums [kMaxStreamCtas][2][16 slots][128 features] fp32 first, the counters after them.
constexpr size_t kStreamPartialBytes = (size_t)kMaxStreamCtas * 2 * 16 * 128 * sizeof(float);
size_t stream_scratch_bytes(int N);
bool stream_supported(int M, int N, int K, int bits, int g);
// `batch_rows` = rows of the whole call this launch is a chunk of (0 = M).  It alone decides between the
// 8-, 16- and 32-row kernel, so that every row of a call goes through the same kernel (and the same
// summation order) whichever chunk it falls into - a routed call moves rows between chunks.
dmr_status_t launch_stream(const uint16_t *X, int M, RowSel sel, const void *weights, const uint16_t *scales,
                           const uint8_t *zeros, int N, int K, int bits, int g, void *Y, dmr_out_t out,
                           void *scratch, int32_t *status, cudaStream_t st, int batch_rows = 0);

// Decode kernel for 4-bit codes (M <= 16 per launch): every CTA owns whole output features and streams their codes
// through warp-private TMA rings; no scratch memory beyond the status word.  sel.idx / sel.count select and
// count the rows of a routed call (the kernel gathers and scatters itself).  `batch_rows` as above.
bool decode_w4_supported(int M, int N, int K, int g);
dmr_status_t launch_decode_w4(const uint16_t *X, int M, RowSel sel, const uint32_t *qweight, const uint16_t *scales,
                              const uint8_t *zeros, int N, int K, int g, void *Y, dmr_out_t out, int32_t *status,
                              cudaStream_t st, int batch_rows = 0);

// The same kernel for 3-bit codes (32 codes in three words): groups and K multiples of 128.
bool decode_w3_supported(int M, int N, int K, int g);
dmr_status_t launch_decode_w3(const uint16_t *X, int M, RowSel sel, const uint32_t *qweight, const uint16_t *scales,
                              const uint8_t *zeros, int N, int K, int g, void *Y, dmr_out_t out, int32_t *status,
                              cudaStream_t st, int batch_rows = 0);

// What the launchers would choose for a call (for dmr_describe_dispatch).
void decode_w4_plan(int M, int g, int *nt, int *r, int *warps);
void decode_w3_plan(int M, int *nt, int *r, int *warps);
void stream_plan(int M, int N, int K, int bits, int *tiles, long long *steps, int *cluster);
void prefill_plan(int M, int N, int K, int *bn, int *splits, long long *tiles, int *ctas);

// Persistent prefill GEMM (M > 32, low-bit weights); sel.idx maps batch slots to rows of X and Y, sel.count
// says how many slots are valid.
bool prefill_supported(int M, int N, int K, int bits, int g);
// X is the caller's activation matrix (for a routed call the rows sel.idx lists are gathered);
// `scratch` holds prefill_scratch_bytes(M, K) bytes for the prepared fp16 activations and their row scales, `partial`
// prefill_partial_bytes(M, N, K) bytes of fp32 partial sums (0 unless the call is split along k).
size_t prefill_scratch_bytes(int M, int K);
size_t prefill_partial_bytes(int M, int N, int K);
dmr_status_t launch_prefill(const uint16_t *X, int M, RowSel sel, const void *qweight, const uint16_t *scales,
                            const uint8_t *zeros, int N, int K, int bits, int g, void *Y, dmr_out_t out,
                            void *scratch, float *partial, int32_t *status, cudaStream_t st);

// Tensor-core GEMM family (M > 16): tcgen05 MMA with TMA-staged operands.
struct GemmPlan {
    int bn;                 // activation rows per CTA (MMA N)
    int splits;             // split-K factor (partials are added in split order)
    int kblocks_per_split;  // 64-wide k blocks per split
    size_t partial_bytes;   // fp32 partial-sum scratch needed (0 when splits == 1)
};
bool gemm_supported(int M, int N, int K, int bits /*0 = bf16 weights*/, int g);
GemmPlan gemm_plan(int M, int N, int K, int bits);
// `weights` is W (bits == 0) or qweight.  X holds M rows (for a routed call: the gathered rows,
// sel.count of them valid); sel.idx maps batch slots to output rows.
dmr_status_t launch_gemm(const uint16_t *X, int M, RowSel sel, const void *weights, const uint16_t *scales,
                         const uint8_t *zeros, int N, int K, int bits, int g, void *Y, dmr_out_t out,
                         float *partial, int32_t *status, cudaStream_t st);
// Y[row(m)][n] = sum over z < splits of partial[z][m][n], in split order (fp32 partial sums by batch slot).
dmr_status_t launch_splitk_reduce(const float *partial, int splits, int M, int N, RowSel sel, void *Y, dmr_out_t out,
                                  cudaStream_t st);
// Xg[s] = X[idx[s]] for the list slots coff <= coff + s < *count (s < Mcap); other slots are zero-filled.
// `idx` is already advanced to slot coff.
dmr_status_t launch_gather_rows(const uint16_t *X, int K, int Mcap, const int32_t *idx, const int32_t *count,
                                int coff, uint16_t *Xg, cudaStream_t st);

// Any-shape fallback (CUDA cores, one warp per output feature).
dmr_status_t launch_simple_lowbit(const uint16_t *X, int M, RowSel sel, const uint32_t *qweight,
                                  const uint16_t *scales, const uint8_t *zeros, int N, int K,
                                  int bits, int g, void *Y, dmr_out_t out, cudaStream_t st);
dmr_status_t launch_simple_dense(const uint16_t *X, int M, RowSel sel, const uint16_t *W, int N,
                                 int K, void *Y, dmr_out_t out, cudaStream_t st);

// Route partition.
dmr_status_t launch_route_partition(const uint8_t *mask, int M, int32_t *idx_high, int32_t *idx_low,
                                    int32_t *counts, cudaStream_t st);

// Step-wise KL divergence: kl_token[i] = KL(softmax(high[i]) || softmax(low[i])) for T rows of V logits
// (bf16 or fp32), kl_step[s] = mean of kl_token over [offsets[s], offsets[s + 1]).
dmr_status_t launch_stepwise_kl(const void *high, const void *low, bool f32, int T, int V, const int32_t *offsets, int S,
                                float *kl_token, float *kl_step, cudaStream_t st);

// Router calibration: tau = the (1 - rho) quantile of `scores` (linear interpolation, binary64); picked: 2 doubles of scratch.
dmr_status_t launch_router_calibrate(const float *scores, int n, double rho, double *tau, double *picked, cudaStream_t st);
dmr_status_t launch_router_mask(const float *scores, int M, const double *tau, uint8_t *mask, cudaStream_t st);

// Router forward (Sec. 4.1): fp32 parameters in the layout dmr.h documents; ws holds router_workspace_bytes().
size_t router_param_floats(const dmr_router_cfg_t &c);
size_t router_workspace_bytes(const dmr_router_cfg_t &c, int B, int L);
size_t router_attention_smem(int L, int dh);
dmr_status_t launch_router_forward(const float *params, const dmr_router_cfg_t &c, const float *Z, const int32_t *lengths, int B,
                                   int L, float *probs, float *scores, int score_class, float *ws, cudaStream_t st);

// One warp waits on a barrier nobody arrives at, with a short limit: *status becomes DMR_ERR_TIMEOUT, *returned 2.
dmr_status_t launch_wait_timeout_selftest(int32_t *status, int32_t *returned, cudaStream_t st);

}  // namespace dmr
