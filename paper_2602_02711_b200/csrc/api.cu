// C ABI of libdmr: argument validation, kernel-family choice and workspace carving.
// Every entry point validates first and launches afterwards; nothing here synchronises the host
// except dmr_workspace_status.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "common.cuh"

namespace dmr {
std::atomic<int> g_last_cuda_error{0};
std::atomic<unsigned long long> g_launches{0};

namespace {

// Workspace layout (all offsets multiples of 256 bytes):
//   [0, 256)   status word
//   routed:    counts {n_high, n_low} (256 B), idx_high [M], idx_low [M]
//   routed, tensor-core path: gathered activations of the low rows [M][K], then of the high rows
//   split-K:   fp32 partial sums [splits][M][N] (shared by the two halves of a routed call)
//   decode:    feature-group counters and per-CTA partial sums of the streaming kernel
struct Scratch {
    int32_t *status = nullptr;
    int32_t *counts = nullptr, *idx_high = nullptr, *idx_low = nullptr;
    uint16_t *xg_low = nullptr, *xg_high = nullptr;
    void *prefill_scratch = nullptr;  // prepared fp16 activations and row scales of the prefill kernel
    float *partial = nullptr;
    void *stream_scratch = nullptr;  // counters + partial sums of the streaming decode kernel
    uint16_t *xg_stream = nullptr;   // routed, decode path: the gathered activation rows of one chunk
    // routed calls run their two halves on two streams: the high-precision half gets its own scratch
    float *partial_high = nullptr;
    void *stream_scratch_high = nullptr;
    uint16_t *xg_stream_high = nullptr;
    size_t bytes = 0;
};

constexpr int kStreamChunk = 32;  // rows one launch of the streaming decode kernel takes at most

// Batches of up to this many rows stay on the streaming decode kernel (in chunks of 32 rows).  The
// default is 32 (two chunks; measured faster than the tensor-core kernels up to there); the environment variable DMR_DECODE_MAX_M moves the crossover for measurements.
int decode_max_m() {
    static int v = -1;
    if (v < 0) {
        const char *e = getenv("DMR_DECODE_MAX_M");
        const int x = e ? atoi(e) : 32;
        v = x < 16 ? 16 : x;
    }
    return v;
}

// The warp-ring decode kernel takes the 4-bit decode batches unless the environment says DMR_DECODE_KERNEL=stream
// (the shared-memory ring kernel, kept for 8-bit codes, bf16 weights and for comparison).
bool decode_w4_enabled() {
    static int v = -1;
    if (v < 0) {
        const char *e = getenv("DMR_DECODE_KERNEL");
        v = (e && strcmp(e, "stream") == 0) ? 0 : 1;
    }
    return v != 0;
}

constexpr int kDecodeChunk = 16;  // rows one launch of the 4-bit decode kernel takes at most

// Whether a call goes to the tensor-core kernels.  For 3-bit codes that family is the persistent prefill kernel alone
// (no split-K kernel): batches it does not take stay on the decode kernel, 16 rows per launch.
bool use_gemm(int M, int N, int K, int bits, int g) {
    if (M <= decode_max_m()) return false;
    if (bits == 3) return prefill_supported(M, N, K, bits, g);
    return gemm_supported(M, N, K, bits, g);
}

Scratch carve(void *workspace, dmr_op_t op, int M, int N, int K, dmr_qformat_t f) {
    Scratch s;
    char *base = reinterpret_cast<char *>(workspace);
    size_t off = kWsStatusBytes;
    s.status = reinterpret_cast<int32_t *>(base);
    const int g = format_ok(K, f) ? group_of(K, f) : K;
    const bool low_gemm = op != DMR_OP_DENSE_LINEAR && use_gemm(M, N, K, f.bits, g);
    const bool dense_gemm = op != DMR_OP_LOWBIT_LINEAR && use_gemm(M, N, K, 0, K);
    if (op == DMR_OP_ROUTED_LINEAR) {
        const size_t list = round_up((size_t)(M > 0 ? M : 1) * 4, 256);
        s.counts = reinterpret_cast<int32_t *>(base + off);
        s.idx_high = reinterpret_cast<int32_t *>(base + off + 256);
        s.idx_low = reinterpret_cast<int32_t *>(base + off + 256 + list);
        off += 256 + 2 * list;
        const size_t xg = round_up((size_t)M * K * 2, 256);
        if (low_gemm) {
            s.xg_low = reinterpret_cast<uint16_t *>(base + off);
            off += xg;
        }
        if (dense_gemm) {
            s.xg_high = reinterpret_cast<uint16_t *>(base + off);
            off += xg;
        }
    }
    if (low_gemm && prefill_supported(M, N, K, f.bits, g)) {
        s.prefill_scratch = base + off;
        off += round_up(prefill_scratch_bytes(M, K), 256);
    }
    const size_t partial_low = !low_gemm ? 0 : (prefill_supported(M, N, K, f.bits, g) ? prefill_partial_bytes(M, N, K) : gemm_plan(M, N, K, f.bits).partial_bytes);
    const size_t partial_dense = dense_gemm ? gemm_plan(M, N, K, 0).partial_bytes : 0;
    if (op == DMR_OP_ROUTED_LINEAR) {
        if (partial_low) {
            s.partial = reinterpret_cast<float *>(base + off);
            off += round_up(partial_low, 256);
        }
        if (partial_dense) {
            s.partial_high = reinterpret_cast<float *>(base + off);
            off += round_up(partial_dense, 256);
        }
    } else if (partial_low || partial_dense) {
        s.partial = reinterpret_cast<float *>(base + off);
        off += round_up(partial_low > partial_dense ? partial_low : partial_dense, 256);
    }
    const bool low_stream = op != DMR_OP_DENSE_LINEAR && !low_gemm;
    const bool dense_stream = op != DMR_OP_LOWBIT_LINEAR && !dense_gemm;
    if (low_stream || dense_stream) {
        s.stream_scratch = base + off;
        off += round_up(stream_scratch_bytes(N), 256);
        if (op == DMR_OP_ROUTED_LINEAR) {
            s.xg_stream = reinterpret_cast<uint16_t *>(base + off);
            off += round_up((size_t)kStreamChunk * K * 2, 256);
            s.stream_scratch_high = base + off;
            off += round_up(stream_scratch_bytes(N), 256);
            s.xg_stream_high = reinterpret_cast<uint16_t *>(base + off);
            off += round_up((size_t)kStreamChunk * K * 2, 256);
        }
    }
    s.bytes = round_up(off, 256);
    return s;
}

dmr_status_t common_checks(const void *X, int M, int N, int K, const void *Y, dmr_out_t out) {
    if (M < 0 || N < 1 || K < 1) return DMR_ERR_INVALID_ARG;
    if (out != DMR_OUT_BF16 && out != DMR_OUT_F32) return DMR_ERR_INVALID_ARG;
    if (M > 0 && (!X || !Y)) return DMR_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(Y)) return DMR_ERR_ALIGNMENT;
    if (K % 8 != 0) return DMR_ERR_UNSUPPORTED;  // rows must be 16-byte multiples
    return DMR_OK;
}

// Rows [0, M) (sel.idx == null) or the listed rows, low-bit weights.  Chooses the kernel family
// from (M, N, K, format) only, never from how many rows a routed call found.
dmr_status_t run_lowbit(const uint16_t *X, int M, RowSel sel, const uint32_t *qweight, const uint16_t *scales,
                        const uint8_t *zeros, int N, int K, dmr_qformat_t f, void *Y, dmr_out_t out,
                        const Scratch &ws, cudaStream_t st) {
    const int g = group_of(K, f);
    const size_t ysz = out == DMR_OUT_F32 ? 4 : 2;
    if (use_gemm(M, N, K, f.bits, g)) {
        if (prefill_supported(M, N, K, f.bits, g))  // gathers the listed rows itself
            return launch_prefill(X, M, sel, qweight, scales, zeros, N, K, f.bits, g, Y, out, ws.prefill_scratch, ws.partial, ws.status, st);
        const uint16_t *Xin = X;
        if (sel.idx) {
            dmr_status_t r = launch_gather_rows(X, K, M, sel.idx, sel.count, 0, ws.xg_low, st);
            if (r != DMR_OK) return r;
            Xin = ws.xg_low;
        }
        return launch_gemm(Xin, M, sel, qweight, scales, zeros, N, K, f.bits, g, Y, out, ws.partial, ws.status, st);
    }
    const bool dec3 = f.bits == 3 && decode_w3_supported(M < kDecodeChunk ? M : kDecodeChunk, N, K, g);
    if (dec3 || (f.bits == 4 && decode_w4_enabled() && decode_w4_supported(M < kDecodeChunk ? M : kDecodeChunk, N, K, g))) {
        // chunks of up to 16 rows; the kernel gathers the rows of a routed call itself
        for (int m0 = 0; m0 < M; m0 += kDecodeChunk) {
            const int mc = M - m0 < kDecodeChunk ? M - m0 : kDecodeChunk;
            RowSel s = sel;
            const uint16_t *Xc = X;
            void *Yc = Y;
            if (sel.idx) {
                s.idx = sel.idx + m0;
                s.offset = sel.offset + m0;
            } else {
                Xc = X + (size_t)m0 * K;
                Yc = reinterpret_cast<char *>(Y) + (size_t)m0 * N * ysz;
            }
            dmr_status_t r = dec3 ? launch_decode_w3(Xc, mc, s, qweight, scales, zeros, N, K, g, Yc, out, ws.status, st, M)
                                  : launch_decode_w4(Xc, mc, s, qweight, scales, zeros, N, K, g, Yc, out, ws.status, st, M);
            if (r != DMR_OK) return r;
        }
        return DMR_OK;
    }
    if (!stream_supported(M < kStreamChunk ? M : kStreamChunk, N, K, f.bits, g))
        return launch_simple_lowbit(X, M, sel, qweight, scales, zeros, N, K, f.bits, g, Y, out, st);
    for (int m0 = 0; m0 < M; m0 += kStreamChunk) {
        const int mc = M - m0 < kStreamChunk ? M - m0 : kStreamChunk;
        RowSel s = sel;
        const uint16_t *Xc = X;
        void *Yc = Y;
        if (sel.idx) {
            s.idx = sel.idx + m0;
            s.offset = sel.offset + m0;
        } else {
            Xc = X + (size_t)m0 * K;
            Yc = reinterpret_cast<char *>(Y) + (size_t)m0 * N * ysz;
        }
        if (sel.idx) {  // the kernel reads consecutive rows: gather this chunk's rows first
            dmr_status_t rg = launch_gather_rows(X, K, mc, s.idx, s.count, s.offset, ws.xg_stream, st);
            if (rg != DMR_OK) return rg;
            Xc = ws.xg_stream;
        }
        dmr_status_t r = launch_stream(Xc, mc, s, qweight, scales, zeros, N, K, f.bits, g, Yc, out, ws.stream_scratch,
                                       ws.status, st, M);
        if (r != DMR_OK) return r;
    }
    return DMR_OK;
}

dmr_status_t run_dense(const uint16_t *X, int M, RowSel sel, const uint16_t *W, int N, int K, void *Y,
                       dmr_out_t out, const Scratch &ws, cudaStream_t st) {
    const size_t ysz = out == DMR_OUT_F32 ? 4 : 2;
    if (use_gemm(M, N, K, 0, K)) {
        const uint16_t *Xin = X;
        if (sel.idx) {
            dmr_status_t r = launch_gather_rows(X, K, M, sel.idx, sel.count, 0, ws.xg_high, st);
            if (r != DMR_OK) return r;
            Xin = ws.xg_high;
        }
        return launch_gemm(Xin, M, sel, W, nullptr, nullptr, N, K, 0, K, Y, out, ws.partial, ws.status, st);
    }
    if (!stream_supported(M < kStreamChunk ? M : kStreamChunk, N, K, 16, K)) return launch_simple_dense(X, M, sel, W, N, K, Y, out, st);
    for (int m0 = 0; m0 < M; m0 += kStreamChunk) {
        const int mc = M - m0 < kStreamChunk ? M - m0 : kStreamChunk;
        RowSel s = sel;
        const uint16_t *Xc = X;
        void *Yc = Y;
        if (sel.idx) {
            s.idx = sel.idx + m0;
            s.offset = sel.offset + m0;
        } else {
            Xc = X + (size_t)m0 * K;
            Yc = reinterpret_cast<char *>(Y) + (size_t)m0 * N * ysz;
        }
        if (sel.idx) {
            dmr_status_t rg = launch_gather_rows(X, K, mc, s.idx, s.count, s.offset, ws.xg_stream, st);
            if (rg != DMR_OK) return rg;
            Xc = ws.xg_stream;
        }
        dmr_status_t r = launch_stream(Xc, mc, s, W, nullptr, nullptr, N, K, 16, K, Yc, out, ws.stream_scratch, ws.status, st, M);
        if (r != DMR_OK) return r;
    }
    return DMR_OK;
}

// Helper stream and fork / join events of the routed call, one set per device, created at the first
// routed call on that device (so make that first call outside any stream capture).
struct SideStream {
    cudaStream_t stream = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
};

// Routed calls of one process enqueue one at a time: the helper stream and its two events are shared per device,
// and a second host thread recording the same events in between would tie the wrong pieces of work together.
std::mutex g_routed_mutex;

SideStream *side_stream() {  // called with g_routed_mutex held
    static SideStream per_device[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    SideStream &s = per_device[dev];
    if (!s.stream) {
        cudaError_t e = cudaStreamCreateWithFlags(&s.stream, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s.fork, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s.join, cudaEventDisableTiming);
        if (e != cudaSuccess) {
            g_last_cuda_error = (int)e;
            s.stream = nullptr;
            return nullptr;
        }
    }
    return &s;
}

}  // namespace
}  // namespace dmr

using namespace dmr;

extern "C" {

size_t dmr_qweight_bytes(int N, int K, dmr_qformat_t f) {
    if (N < 1 || !format_ok(K, f)) return 0;
    return (size_t)N * K * f.bits / 8;
}

size_t dmr_scales_bytes(int N, int K, dmr_qformat_t f) {
    if (N < 1 || !format_ok(K, f)) return 0;
    return (size_t)N * (K / group_of(K, f)) * 2;
}

size_t dmr_zeros_bytes(int N, int K, dmr_qformat_t f) {
    if (N < 1 || !format_ok(K, f)) return 0;
    return (size_t)N * (K / group_of(K, f));
}

size_t dmr_workspace_bytes(dmr_op_t op, int M, int N, int K, dmr_qformat_t f) {
    if (M < 0 || N < 1 || K < 1) return kWsStatusBytes;
    return carve(nullptr, op, M, N, K, f).bytes;
}

dmr_status_t dmr_quantize(const void *W_bf16, int N, int K, dmr_qformat_t f, void *qweight, void *scales,
                          void *zeros, int32_t *dev_status, void *stream) {
    if (N < 1 || K < 1 || !W_bf16 || !qweight || !scales || !zeros) return DMR_ERR_INVALID_ARG;
    if (f.bits != 3 && f.bits != 4 && f.bits != 8) return DMR_ERR_UNSUPPORTED;
    if (!format_ok(K, f)) return DMR_ERR_INVALID_ARG;
    if (!aligned16(W_bf16) || !aligned16(qweight)) return DMR_ERR_ALIGNMENT;
    return launch_quantize(reinterpret_cast<const uint16_t *>(W_bf16), N, K, f.bits, group_of(K, f),
                           reinterpret_cast<uint32_t *>(qweight), reinterpret_cast<uint16_t *>(scales),
                           reinterpret_cast<uint8_t *>(zeros), dev_status, (cudaStream_t)stream);
}

dmr_status_t dmr_dequantize(const void *qweight, const void *scales, const void *zeros, int N, int K,
                            dmr_qformat_t f, void *W_out, dmr_out_t out, void *stream) {
    if (N < 1 || K < 1 || !qweight || !scales || !zeros || !W_out) return DMR_ERR_INVALID_ARG;
    if (out != DMR_OUT_BF16 && out != DMR_OUT_F32) return DMR_ERR_INVALID_ARG;
    if (f.bits != 3 && f.bits != 4 && f.bits != 8) return DMR_ERR_UNSUPPORTED;
    if (!format_ok(K, f)) return DMR_ERR_INVALID_ARG;
    if (!aligned16(qweight) || !aligned16(W_out)) return DMR_ERR_ALIGNMENT;
    return launch_dequantize(reinterpret_cast<const uint32_t *>(qweight), reinterpret_cast<const uint16_t *>(scales),
                             reinterpret_cast<const uint8_t *>(zeros), N, K, f.bits, group_of(K, f), W_out, out,
                             (cudaStream_t)stream);
}

dmr_status_t dmr_lowbit_linear(const void *X_bf16, int M, const void *qweight, const void *scales,
                               const void *zeros, int N, int K, dmr_qformat_t f, void *Y, dmr_out_t out,
                               void *workspace, size_t workspace_bytes, void *stream) {
    dmr_status_t r = common_checks(X_bf16, M, N, K, Y, out);
    if (r != DMR_OK) return r;
    if (!qweight || !scales || !zeros) return DMR_ERR_INVALID_ARG;
    if (f.bits != 3 && f.bits != 4 && f.bits != 8) return DMR_ERR_UNSUPPORTED;
    if (!format_ok(K, f)) return DMR_ERR_INVALID_ARG;
    if (!aligned16(qweight)) return DMR_ERR_ALIGNMENT;
    if (M == 0) return DMR_OK;  // nothing to do, no workspace needed
    if (!workspace || workspace_bytes < dmr_workspace_bytes(DMR_OP_LOWBIT_LINEAR, M, N, K, f)) return DMR_ERR_WORKSPACE;
    if (!aligned16(workspace)) return DMR_ERR_ALIGNMENT;
    RowSel sel = {nullptr, nullptr, 0};
    const Scratch ws = carve(workspace, DMR_OP_LOWBIT_LINEAR, M, N, K, f);
    return run_lowbit(reinterpret_cast<const uint16_t *>(X_bf16), M, sel, reinterpret_cast<const uint32_t *>(qweight),
                      reinterpret_cast<const uint16_t *>(scales), reinterpret_cast<const uint8_t *>(zeros), N, K, f,
                      Y, out, ws, (cudaStream_t)stream);
}

dmr_status_t dmr_dense_linear(const void *X_bf16, int M, const void *W_bf16, int N, int K, void *Y,
                              dmr_out_t out, void *workspace, size_t workspace_bytes, void *stream) {
    dmr_status_t r = common_checks(X_bf16, M, N, K, Y, out);
    if (r != DMR_OK) return r;
    if (!W_bf16) return DMR_ERR_INVALID_ARG;
    if (!aligned16(W_bf16)) return DMR_ERR_ALIGNMENT;
    dmr_qformat_t f = {4, 0};
    if (M == 0) return DMR_OK;  // nothing to do, no workspace needed
    if (!workspace || workspace_bytes < dmr_workspace_bytes(DMR_OP_DENSE_LINEAR, M, N, K, f)) return DMR_ERR_WORKSPACE;
    if (!aligned16(workspace)) return DMR_ERR_ALIGNMENT;
    RowSel sel = {nullptr, nullptr, 0};
    const Scratch ws = carve(workspace, DMR_OP_DENSE_LINEAR, M, N, K, f);
    return run_dense(reinterpret_cast<const uint16_t *>(X_bf16), M, sel, reinterpret_cast<const uint16_t *>(W_bf16), N,
                     K, Y, out, ws, (cudaStream_t)stream);
}

dmr_status_t dmr_route_partition(const uint8_t *mask, int M, int32_t *idx_high, int32_t *idx_low,
                                 int32_t *counts, void *stream) {
    if (M < 0 || !counts) return DMR_ERR_INVALID_ARG;
    if (M > 0 && (!mask || !idx_high || !idx_low)) return DMR_ERR_INVALID_ARG;
    return launch_route_partition(mask, M, idx_high, idx_low, counts, (cudaStream_t)stream);
}

dmr_status_t dmr_routed_linear(const void *X_bf16, int M, const uint8_t *mask, const void *W_bf16,
                               const void *qweight, const void *scales, const void *zeros, int N, int K,
                               dmr_qformat_t f, void *Y, dmr_out_t out, void *workspace,
                               size_t workspace_bytes, void *stream) {
    dmr_status_t r = common_checks(X_bf16, M, N, K, Y, out);
    if (r != DMR_OK) return r;
    if (!W_bf16 || !qweight || !scales || !zeros) return DMR_ERR_INVALID_ARG;
    if (M > 0 && !mask) return DMR_ERR_INVALID_ARG;
    if (f.bits != 3 && f.bits != 4 && f.bits != 8) return DMR_ERR_UNSUPPORTED;
    if (!format_ok(K, f)) return DMR_ERR_INVALID_ARG;
    if (!aligned16(W_bf16) || !aligned16(qweight)) return DMR_ERR_ALIGNMENT;
    if (M == 0) return DMR_OK;  // nothing to do, no workspace needed
    if (!workspace || workspace_bytes < dmr_workspace_bytes(DMR_OP_ROUTED_LINEAR, M, N, K, f)) return DMR_ERR_WORKSPACE;
    if (!aligned16(workspace)) return DMR_ERR_ALIGNMENT;
    cudaStream_t st = (cudaStream_t)stream;
    const Scratch ws = carve(workspace, DMR_OP_ROUTED_LINEAR, M, N, K, f);
    std::lock_guard<std::mutex> routed_lock(g_routed_mutex);
    r = launch_route_partition(mask, M, ws.idx_high, ws.idx_low, ws.counts, st);
    if (r != DMR_OK) return r;
    const uint16_t *X = reinterpret_cast<const uint16_t *>(X_bf16);
    // the two halves touch different rows of Y and different scratch: the high-precision half runs on a
    // helper stream, forked after the partition and joined before the call's work on `stream` ends
    SideStream *side = side_stream();
    if (!side) return DMR_ERR_CUDA;
    cudaError_t e = cudaEventRecord(side->fork, st);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(side->stream, side->fork, 0);
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        return DMR_ERR_CUDA;
    }
    Scratch wh = ws;
    wh.partial = ws.partial_high;
    wh.stream_scratch = ws.stream_scratch_high;
    wh.xg_stream = ws.xg_stream_high;
    RowSel high = {ws.idx_high, ws.counts + 0, 0};
    const dmr_status_t rh = run_dense(X, M, high, reinterpret_cast<const uint16_t *>(W_bf16), N, K, Y, out, wh, side->stream);
    RowSel low = {ws.idx_low, ws.counts + 1, 0};
    const dmr_status_t rl = run_lowbit(X, M, low, reinterpret_cast<const uint32_t *>(qweight), reinterpret_cast<const uint16_t *>(scales),
                                       reinterpret_cast<const uint8_t *>(zeros), N, K, f, Y, out, ws, st);
    // always join, also after an error, so that the helper stream never outlives the call (or a capture)
    e = cudaEventRecord(side->join, side->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, side->join, 0);
    if (rh != DMR_OK) return rh;
    if (rl != DMR_OK) return rl;
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        return DMR_ERR_CUDA;
    }
    return DMR_OK;
}

size_t dmr_host_staging_bytes(int M, int N, int K, dmr_out_t out) {
    if (M < 0 || N < 1 || K < 1) return 0;
    return round_up((size_t)M * K * 2, 256) + round_up((size_t)M * N * (out == DMR_OUT_F32 ? 4 : 2), 256) + 256;
}

dmr_status_t dmr_lowbit_linear_host(const void *X_host, int M, const void *qweight, const void *scales,
                                    const void *zeros, int N, int K, dmr_qformat_t f, void *Y_host,
                                    dmr_out_t out, void *staging, size_t staging_bytes, void *workspace,
                                    size_t workspace_bytes, void *stream) {
    if (M < 0 || N < 1 || K < 1) return DMR_ERR_INVALID_ARG;
    if (M > 0 && (!X_host || !Y_host)) return DMR_ERR_INVALID_ARG;
    if (!staging || staging_bytes < dmr_host_staging_bytes(M, N, K, out)) return DMR_ERR_WORKSPACE;
    if (!aligned16(staging)) return DMR_ERR_ALIGNMENT;
    if (M == 0) return DMR_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t xbytes = (size_t)M * K * 2, ybytes = (size_t)M * N * (out == DMR_OUT_F32 ? 4 : 2);
    char *Xd = reinterpret_cast<char *>(staging);
    char *Yd = Xd + round_up(xbytes, 256);
    cudaError_t e = cudaMemcpyAsync(Xd, X_host, xbytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        return DMR_ERR_CUDA;
    }
    dmr_status_t r = dmr_lowbit_linear(Xd, M, qweight, scales, zeros, N, K, f, Yd, out, workspace, workspace_bytes, stream);
    if (r != DMR_OK) return r;
    e = cudaMemcpyAsync(Y_host, Yd, ybytes, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        return DMR_ERR_CUDA;
    }
    return DMR_OK;
}

dmr_status_t dmr_stepwise_kl(const void *logits_high, const void *logits_low, dmr_out_t dtype, int T, int V,
                             const int32_t *step_offsets, int S, float *kl_token, float *kl_step, void *stream) {
    if (T < 0 || V < 1 || S < 0) return DMR_ERR_INVALID_ARG;
    if (dtype != DMR_OUT_BF16 && dtype != DMR_OUT_F32) return DMR_ERR_INVALID_ARG;
    if (T > 0 && (!logits_high || !logits_low || !kl_token)) return DMR_ERR_INVALID_ARG;
    if (S > 0 && (!step_offsets || !kl_step)) return DMR_ERR_INVALID_ARG;
    if (!aligned16(logits_high) || !aligned16(logits_low)) return DMR_ERR_ALIGNMENT;
    if (T == 0 && S == 0) return DMR_OK;
    return launch_stepwise_kl(logits_high, logits_low, dtype == DMR_OUT_F32, T, V, step_offsets, S, kl_token, kl_step,
                              reinterpret_cast<cudaStream_t>(stream));
}

dmr_status_t dmr_workspace_status(const void *workspace, void *stream) {
    if (!workspace) return DMR_ERR_INVALID_ARG;
    int32_t v = 0;
    cudaError_t e = cudaMemcpyAsync(&v, workspace, sizeof v, cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        return DMR_ERR_CUDA;
    }
    return v == 0 ? DMR_OK : (dmr_status_t)v;
}

int dmr_describe_dispatch(dmr_op_t op, int M, int N, int K, dmr_qformat_t f, char *buf, size_t buf_bytes) {
    if (!buf || buf_bytes == 0 || M < 1 || N < 1 || K < 1) return -1;
    const bool dense = op == DMR_OP_DENSE_LINEAR;
    if (op != DMR_OP_LOWBIT_LINEAR && op != DMR_OP_DENSE_LINEAR) return -1;
    if (!dense && !format_ok(K, f)) return -1;
    const int bits = dense ? 0 : f.bits, g = dense ? K : group_of(K, f);
    if (use_gemm(M, N, K, bits, g)) {
        if (!dense && prefill_supported(M, N, K, bits, g)) {
            int bn, splits, ctas;
            long long tiles;
            prefill_plan(M, N, K, &bn, &splits, &tiles, &ctas);
            return snprintf(buf, buf_bytes, "prefill bits=%d bn=%d splits=%d tiles=%lld ctas=%d", bits, bn, splits, tiles, ctas);
        }
        const GemmPlan p = gemm_plan(M, N, K, bits);
        return snprintf(buf, buf_bytes, "gemm bits=%d bn=%d splits=%d", bits, p.bn, p.splits);
    }
    if (!dense && bits == 3 && decode_w3_supported(M < kDecodeChunk ? M : kDecodeChunk, N, K, g)) {
        int nt, r, warps;
        decode_w3_plan(M, &nt, &r, &warps);
        return snprintf(buf, buf_bytes, "decode_w3 rows=%d tile=%d warps=%d chunks=%d", 8 * nt, 16 * r, warps, (M + kDecodeChunk - 1) / kDecodeChunk);
    }
    if (!dense && bits == 4 && decode_w4_enabled() && decode_w4_supported(M < kDecodeChunk ? M : kDecodeChunk, N, K, g)) {
        int nt, r, warps;
        decode_w4_plan(M, g, &nt, &r, &warps);
        return snprintf(buf, buf_bytes, "decode_w4 rows=%d tile=%d warps=%d chunks=%d", 8 * nt, 16 * r, warps, (M + kDecodeChunk - 1) / kDecodeChunk);
    }
    const int sbits = dense ? 16 : bits;
    if (!stream_supported(M < kStreamChunk ? M : kStreamChunk, N, K, sbits, g)) return snprintf(buf, buf_bytes, "simple bits=%d", sbits);
    int tiles, cluster;
    long long steps;
    stream_plan(M < kStreamChunk ? M : kStreamChunk, N, K, sbits, &tiles, &steps, &cluster);
    return snprintf(buf, buf_bytes, "stream bits=%d rows=%d steps=%lld cluster=%d chunks=%d", sbits, 8 * tiles, steps, cluster,
                    (M + kStreamChunk - 1) / kStreamChunk);
}

static bool router_cfg_ok(const dmr_router_cfg_t &c) {
    if (c.d < 16 || c.d > 1024 || c.d % 16 != 0) return false;
    if (c.heads < 1 || c.d % c.heads != 0) return false;
    if (c.ffn < 16 || c.ffn % 16 != 0 || c.ffn > 65536) return false;
    if (c.layers < 1 || c.layers > 64) return false;
    if (c.l_max < 1 || c.l_max > 128) return false;
    if (c.classes < 1 || c.classes > 32) return false;
    return router_attention_smem(c.l_max, c.d / c.heads) <= 200 * 1024;
}

size_t dmr_router_param_floats(dmr_router_cfg_t cfg) { return router_cfg_ok(cfg) ? router_param_floats(cfg) : 0; }

size_t dmr_router_workspace_bytes(dmr_router_cfg_t cfg, int B, int L) {
    if (!router_cfg_ok(cfg) || B < 1 || L < 1 || L > cfg.l_max) return 0;
    return router_workspace_bytes(cfg, B, L);
}

dmr_status_t dmr_router_forward(const float *params, dmr_router_cfg_t cfg, const float *Z, const int32_t *lengths, int B,
                                int L, float *probs, float *scores, int score_class, void *workspace,
                                size_t workspace_bytes, void *stream) {
    if (!router_cfg_ok(cfg) || B < 0 || L < 1 || L > cfg.l_max) return DMR_ERR_INVALID_ARG;
    if ((long long)B * L > (1ll << 24)) return DMR_ERR_UNSUPPORTED;
    if (scores && (score_class < 0 || score_class >= cfg.classes)) return DMR_ERR_INVALID_ARG;
    if (B == 0) return DMR_OK;
    if (!params || !Z || !lengths || !probs) return DMR_ERR_INVALID_ARG;
    if (!aligned16(params) || !aligned16(Z)) return DMR_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < router_workspace_bytes(cfg, B, L)) return DMR_ERR_WORKSPACE;
    if (!aligned16(workspace)) return DMR_ERR_ALIGNMENT;
    return launch_router_forward(params, cfg, Z, lengths, B, L, probs, scores, score_class, reinterpret_cast<float *>(workspace),
                                 (cudaStream_t)stream);
}

dmr_status_t dmr_router_calibrate(const float *cal_scores, int n, double rho, double *tau, void *stream) {
    if (!cal_scores || !tau || n < 1) return DMR_ERR_INVALID_ARG;
    if (!(rho >= 0.0 && rho <= 1.0)) return DMR_ERR_INVALID_ARG;
    if (n > 65536) return DMR_ERR_UNSUPPORTED;
    if (((uintptr_t)tau & 15u) != 0) return DMR_ERR_ALIGNMENT;  // tau[0] is the result, tau[1..2] scratch
    return launch_router_calibrate(cal_scores, n, rho, tau, tau + 1, (cudaStream_t)stream);
}

dmr_status_t dmr_router_mask(const float *scores, int M, const double *tau, uint8_t *mask, void *stream) {
    if (M < 0 || !tau) return DMR_ERR_INVALID_ARG;
    if (M == 0) return DMR_OK;
    if (!scores || !mask) return DMR_ERR_INVALID_ARG;
    return launch_router_mask(scores, M, tau, mask, (cudaStream_t)stream);
}

dmr_status_t dmr_selftest_wait_timeout(void *workspace, size_t workspace_bytes, void *stream) {
    if (!workspace || workspace_bytes < kWsStatusBytes) return DMR_ERR_WORKSPACE;
    if (!aligned16(workspace)) return DMR_ERR_ALIGNMENT;
    int32_t *w = reinterpret_cast<int32_t *>(workspace);
    return launch_wait_timeout_selftest(w, w + 1, (cudaStream_t)stream);
}

const char *dmr_status_string(dmr_status_t s) {
    switch (s) {
        case DMR_OK: return "ok";
        case DMR_ERR_INVALID_ARG: return "invalid argument";
        case DMR_ERR_UNSUPPORTED: return "unsupported format or shape";
        case DMR_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case DMR_ERR_WORKSPACE: return "workspace missing or too small";
        case DMR_ERR_NONFINITE: return "non-finite weight";
        case DMR_ERR_TIMEOUT: return "bounded wait ran out on the device";
        case DMR_ERR_CUDA: return "CUDA error";
    }
    return "unknown status";
}

int dmr_last_cuda_error(void) { return g_last_cuda_error; }

uint64_t dmr_launch_count(void) { return g_launches; }

}  // extern "C"
