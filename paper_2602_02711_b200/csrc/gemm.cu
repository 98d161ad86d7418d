// Tensor-core GEMM family (M > 16): prefill-sized low-bit linear layers, the dense bf16 linear of
// the high-precision rows, and the routed batch.  The product is a dense contraction, so it runs
// on tcgen05: operands staged in shared memory by TMA, fp32 accumulators in tensor memory.
//
// Orientation.  The weights are the 128-row operand of the MMA and the activation rows are its
// N operand (D[n][m] = sum_k W[n][k] X[m][k]), so one tensor-memory lane holds one output feature.
// That puts the per-(feature, group) scale on a lane: the low-bit path feeds the tensor core the
// exact integers q - zero, lets it sum one quantization group into a tensor-memory buffer, and the
// scale warps multiply that group sum by the feature's bf16 scale while adding it to fp32
// accumulators in registers (two buffers, so the next group's MMAs overlap).  No weight is rounded;
// the result differs from exact arithmetic by fp32 summation only.
//
// Warps: 0 = TMA producer, 1 = MMA issuer (owns tensor memory), 2..5 = unpack warps (low-bit:
// packed tile -> swizzled bf16 A tile; one thread per feature row), 6..9 = scale/epilogue warps
// (dense: warps 2..5 are the epilogue).  All waits are bounded.
#include <cuda_bf16.h>

#include "sm100.cuh"

namespace dmr {

namespace {

constexpr int BM = 128;  // features per CTA (MMA M)
constexpr int BK = 64;   // k per stage: one 128-byte swizzled row of bf16

template <int MODE, int BN>
struct GemmCfg {
    static constexpr int A_BYTES = BM * BK * 2;                        // 16 KB
    static constexpr int B_BYTES = BN * BK * 2;
    static constexpr int P_ROW = MODE == 0 ? 0 : BK * MODE / 8;         // packed bytes per row per stage
    static constexpr int P_BYTES = ((BM * P_ROW + 1023) / 1024) * 1024;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + P_BYTES;
    static constexpr int STAGES_RAW = (200 * 1024) / STAGE_BYTES;
    static constexpr int STAGES = STAGES_RAW > 8 ? 8 : STAGES_RAW;
    static constexpr int THREADS = MODE == 0 ? 192 : 320;
    static constexpr int TMEM_COLS_RAW = MODE == 0 ? BN : 2 * BN;
    static constexpr int TMEM_COLS = TMEM_COLS_RAW < 32 ? 32 : TMEM_COLS_RAW;
    static constexpr size_t SMEM = (size_t)STAGES * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;
};

struct GemmArgs {
    const uint16_t *scales;   // low-bit only
    const uint8_t *zeros;     // low-bit only
    void *Y;                  // [M][N] output, or nullptr when writing split-K partials
    float *partial;           // [splits][Mrows][N] fp32 partial sums (split-K), else nullptr
    const int32_t *idx;       // routed: output row of batch slot m (nullptr = identity)
    const int32_t *count;     // routed: number of valid slots (nullptr = M)
    int32_t *status;
    int M, N, K, g_size, kblocks_per_split;
};


template <int MODE, int BN, bool OUT_F32>
__global__ void __launch_bounds__(GemmCfg<MODE, BN>::THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, GemmArgs args) {
    using Cfg = GemmCfg<MODE, BN>;
    constexpr int S = Cfg::STAGES;
    constexpr bool LOWBIT = MODE != 0;
    extern __shared__ uint8_t smem_dyn[];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * BM;
    const int m0 = blockIdx.y * BN;
    const int split = blockIdx.z;
    const int rows = args.count ? min(*args.count, args.M) : args.M;
    if (m0 >= rows) return;  // routed: this column block holds no row (uniform across the CTA)

    const int kb_total = args.K / BK;
    const int kb_begin = split * args.kblocks_per_split;
    const int kb_end = min(kb_total, kb_begin + args.kblocks_per_split);
    const int nkb = kb_end - kb_begin;  // >= 1 by construction of the grid

    // ---- shared memory carve-up (tiles 1024-byte aligned for the 128-byte swizzle) ----
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
    auto a_tile = [&](int s) { return base + s * Cfg::STAGE_BYTES; };
    auto b_tile = [&](int s) { return base + s * Cfg::STAGE_BYTES + Cfg::A_BYTES; };
    auto p_tile = [&](int s) { return base + s * Cfg::STAGE_BYTES + Cfg::A_BYTES + Cfg::B_BYTES; };
    const uint32_t bar_base = base + S * Cfg::STAGE_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8 * s; };
    auto empty_bar = [&](int s) { return bar_base + 64 + 8 * s; };
    auto ready_bar = [&](int s) { return bar_base + 128 + 8 * s; };
    auto tfull_bar = [&](int b) { return bar_base + 192 + 8 * b; };
    auto tempty_bar = [&](int b) { return bar_base + 208 + 8 * b; };
    const uint32_t tmem_slot = bar_base + 224;
    volatile uint32_t *tmem_slot_ptr = reinterpret_cast<volatile uint32_t *>(base_ptr + S * Cfg::STAGE_BYTES + 224);

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
            mbar_init(ready_bar(s), 128);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), 128);
        }
        fence_barrier_init();
        prefetch_tensor_map(&map_w);
        prefetch_tensor_map(&map_x);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
        tmem_relinquish();
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot_ptr;

    // Set-up done: only now wait for the kernels before this one (gathered rows, row lists), and let the kernel behind
    // this one start its own set-up.
    pdl_wait();
    pdl_launch_dependents();
    // quantization groups seen by this CTA: group boundaries in units of k-blocks
    const int kb_per_group = LOWBIT ? max(1, args.g_size / BK) : kb_total;

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            constexpr uint32_t TX = Cfg::B_BYTES + (LOWBIT ? BM * Cfg::P_ROW : Cfg::A_BYTES);
            for (int i = 0; i < nkb; ++i) {
                const int s = i % S;
                if (i >= S && !mbar_wait(empty_bar(s), (uint32_t)(((i / S) - 1) & 1), args.status)) break;
                const int kb = kb_begin + i;
                mbar_expect_tx(full_bar(s), TX);
                tma_load_2d(b_tile(s), &map_x, full_bar(s), kb * BK, m0);
                if (LOWBIT) tma_load_2d(p_tile(s), &map_w, full_bar(s), kb * Cfg::P_ROW, n0);
                else tma_load_2d(a_tile(s), &map_w, full_bar(s), kb * BK, n0);
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        // the whole warp runs the loop (the same stage numbers and descriptors in all lanes), one lane issues
        {
            constexpr uint32_t IDESC = umma_idesc_bf16(BM, BN);
            // operand descriptors of stage 0; a stage and a k step only move the address field (16-byte units)
            const uint64_t desc_a0 = umma_desc_sw128(a_tile(0)), desc_b0 = umma_desc_sw128(b_tile(0));
            int buf = 0, groups_done = 0;
            bool group_start = true;
            for (int i = 0; i < nkb; ++i) {
                const int s = i % S;
                const uint32_t par = (uint32_t)((i / S) & 1);
                if (!mbar_wait(full_bar(s), par, args.status)) break;
                if (LOWBIT && !mbar_wait(ready_bar(s), par, args.status)) break;
                if (LOWBIT && group_start && groups_done >= 2) {
                    // the scale warps must have drained this buffer's previous group
                    if (!mbar_wait(tempty_bar(buf), (uint32_t)(((groups_done >> 1) - 1) & 1), args.status)) break;
                }
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                const uint64_t stage_off = (uint64_t)(((uint32_t)s * (uint32_t)Cfg::STAGE_BYTES) >> 4);
                if (lane == 0) {
#pragma unroll
                    for (int j = 0; j < BK / 16; ++j)  // 16 k values = 32 bytes of a row = two 16-byte units
                        umma_bf16_ss(d_tmem, desc_a0 + stage_off + (uint64_t)(2 * j), desc_b0 + stage_off + (uint64_t)(2 * j), IDESC,
                                     (group_start && j == 0) ? 0u : 1u);
                    umma_commit(empty_bar(s));
                }
                __syncwarp();
                group_start = false;
                const int kb = kb_begin + i;
                const bool group_end = LOWBIT ? (((kb + 1) % kb_per_group) == 0 || i == nkb - 1) : (i == nkb - 1);
                if (group_end) {
                    if (lane == 0) umma_commit(tfull_bar(buf));
                    __syncwarp();
                    if (LOWBIT) buf ^= 1;
                    ++groups_done;
                    group_start = true;
                }
            }
        }
    } else if (LOWBIT && warp < 6) {
        // ================= unpack warps: packed codes -> exact integers (q - zero) as bf16 =================
        const int r = (warp - 2) * 32 + lane;   // feature row of the tile
        const int n = min(n0 + r, args.N - 1);
        const int G = args.K / args.g_size;
        const uint32_t swz = (uint32_t)(r & 7);
        for (int i = 0; i < nkb; ++i) {
            const int s = i % S;
            const int kb = kb_begin + i;
            const uint32_t zb = __ldg(args.zeros + (size_t)n * G + (kb * BK) / args.g_size);
            if (!mbar_wait(full_bar(s), (uint32_t)((i / S) & 1), args.status)) break;
            const uint32_t src = p_tile(s) + r * Cfg::P_ROW;
            const uint32_t dst = a_tile(s) + r * 128;
            if (MODE == 4) {
                uint32_t w[8];
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(src));
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]) : "r"(src + 16));
                const uint32_t zz = 0x4300u | zb;
                const uint32_t zoff = zz | (zz << 16);
#pragma unroll
                for (int c = 0; c < 8; ++c) {  // word c = codes 8c .. 8c+7 = 16-byte chunk c of the row
                    const uint32_t d04 = bf16x2_sub(lop3_and_or(w[c], 0x000F000Fu, 0x43004300u), zoff);
                    const uint32_t d15 = bf16x2_sub(lop3_and_or(w[c] >> 4, 0x000F000Fu, 0x43004300u), zoff);
                    const uint32_t d26 = bf16x2_sub(lop3_and_or(w[c] >> 8, 0x000F000Fu, 0x43004300u), zoff);
                    const uint32_t d37 = bf16x2_sub(lop3_and_or(w[c] >> 12, 0x000F000Fu, 0x43004300u), zoff);
                    const uint32_t o01 = prmt(d04, d15, 0x5410), o45 = prmt(d04, d15, 0x7632);
                    const uint32_t o23 = prmt(d26, d37, 0x5410), o67 = prmt(d26, d37, 0x7632);
                    const uint32_t addr = dst + ((((uint32_t)c) ^ swz) << 4);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(o01), "r"(o23), "r"(o45), "r"(o67) : "memory");
                }
            } else {
                const float zf = __uint_as_float(0x4B000000u | zb);
#pragma unroll
                for (int c = 0; c < 8; ++c) {  // chunk c = codes 8c .. 8c+7 = packed words 2c, 2c+1
                    uint32_t w0, w1;
                    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(w0), "=r"(w1) : "r"(src + 8 * c));
                    uint32_t o[4];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint32_t u = h ? w1 : w0;
                        float f[4];
#pragma unroll
                        for (int b = 0; b < 4; ++b)
                            f[b] = __fsub_rn(__uint_as_float(prmt(u, 0x4B000000u, 0x7650u + (uint32_t)b)), zf);
                        o[2 * h] = pack_bf16x2_rn(f[0], f[1]);
                        o[2 * h + 1] = pack_bf16x2_rn(f[2], f[3]);
                    }
                    const uint32_t addr = dst + ((((uint32_t)c) ^ swz) << 4);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
                }
            }
            fence_proxy_async_smem();  // make the tile visible to the tensor core's reads
            mbar_arrive(ready_bar(s));
        }
    } else {
        // ================= scale / epilogue warps =================
        const int q = warp & 3;                  // tensor-memory lane quadrant this warp may read
        const int r = q * 32 + lane;             // feature row of the tile
        const int n = n0 + r;
        const int nc = min(n, args.N - 1);
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        const int G = LOWBIT ? args.K / args.g_size : 1;
        (void)nc;
        (void)G;
        // groups this CTA sums: from the group containing kb_begin to the one containing kb_end - 1
        const int ngroups = LOWBIT ? ((kb_end - 1) / kb_per_group - kb_begin / kb_per_group + 1) : 1;
        auto store16 = [&](int c0, const float (&v)[16]) {
            if (n >= args.N) return;
            if (args.partial) {
                float *dst = args.partial + ((size_t)split * args.M + m0 + c0) * args.N + n;
#pragma unroll
                for (int c = 0; c < 16; ++c)
                    if (m0 + c0 + c < rows) dst[(size_t)c * args.N] = v[c];
            } else {
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const int m = m0 + c0 + c;
                    if (m < rows) {
                        const int row = args.idx ? args.idx[m] : m;
                        if (OUT_F32) reinterpret_cast<float *>(args.Y)[(size_t)row * args.N + n] = v[c];
                        else reinterpret_cast<__nv_bfloat16 *>(args.Y)[(size_t)row * args.N + n] = __float2bfloat16_rn(v[c]);
                    }
                }
            }
        };
        if (LOWBIT) {
            constexpr int ACC = LOWBIT ? BN : 16;
            float acc[ACC];
#pragma unroll
            for (int c = 0; c < ACC; ++c) acc[c] = 0.f;
            bool ok = true;
            for (int gi = 0; gi < ngroups && ok; ++gi) {
                const int buf = gi & 1;
                const int grp = kb_begin / kb_per_group + gi;
                const float sc = __uint_as_float((uint32_t)__ldg(args.scales + (size_t)nc * G + grp) << 16);
                ok = mbar_wait(tfull_bar(buf), (uint32_t)((gi >> 1) & 1), args.status);
                if (!ok) break;
                tcgen05_fence_after();
#pragma unroll
                for (int c0 = 0; c0 < ACC; c0 += 16) {
                    uint32_t v[16];
                    tmem_ld_x16(lane_addr + (uint32_t)(buf * BN + c0), v);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 16; ++c) acc[c0 + c] = fmaf(sc, __uint_as_float(v[c]), acc[c0 + c]);
                }
                tcgen05_fence_before();
                mbar_arrive(tempty_bar(buf));
            }
            if (ok) {
#pragma unroll
                for (int c0 = 0; c0 < ACC; c0 += 16) {
                    float v[16];
#pragma unroll
                    for (int c = 0; c < 16; ++c) v[c] = acc[c0 + c];
                    store16(c0, v);
                }
            }
        } else {
            if (mbar_wait(tfull_bar(0), 0, args.status)) {
                tcgen05_fence_after();
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 16) {
                    if (m0 + c0 >= rows) break;
                    uint32_t u[16];
                    tmem_ld_x16(lane_addr + (uint32_t)c0, u);
                    tmem_ld_wait();
                    float v[16];
#pragma unroll
                    for (int c = 0; c < 16; ++c) v[c] = __uint_as_float(u[c]);
                    store16(c0, v);
                }
            }
        }
    }

    // ---- teardown: every role's loop is bounded, so all warps arrive here ----
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after();
        tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
    }
}

// Split-K: Y[row(m)][n] = sum over splits, in split order.
template <bool OUT_F32>
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float *__restrict__ partial, int splits, int M, int N, const int32_t *__restrict__ idx,
                     const int32_t *__restrict__ count, void *__restrict__ Y) {
    pdl_wait();  // the partial sums come from the kernel before this one
    pdl_launch_dependents();
    const int rows = count ? min(*count, M) : M;
    if ((N & 3) == 0 && (size_t)rows * (size_t)N < 0x7FFFFFFFull) {
        // four consecutive features per thread: 16-byte loads of every split's sums, one 8- or 16-byte store
        const unsigned nq = (unsigned)N >> 2, total = (unsigned)rows * nq;
        const size_t zstride = (size_t)M * (size_t)N / 4;
        for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
            const unsigned m = i / nq, q = i - m * nq;
            const int row = idx ? idx[m] : (int)m;
            const float4 *p = reinterpret_cast<const float4 *>(partial) + (size_t)m * nq + q;
            float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int z = 0; z < splits; ++z) {  // in split order, as the one-element path below
                const float4 v = p[(size_t)z * zstride];
                s.x += v.x;
                s.y += v.y;
                s.z += v.z;
                s.w += v.w;
            }
            const size_t o = (size_t)row * N + 4u * q;
            if (OUT_F32) {
                *reinterpret_cast<float4 *>(reinterpret_cast<float *>(Y) + o) = s;
            } else {
                const __nv_bfloat162 lo = __floats2bfloat162_rn(s.x, s.y), hi = __floats2bfloat162_rn(s.z, s.w);
                uint2 w;
                w.x = *reinterpret_cast<const uint32_t *>(&lo);
                w.y = *reinterpret_cast<const uint32_t *>(&hi);
                *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(Y) + o) = w;
            }
        }
        return;
    }
    const size_t total = (size_t)rows * N;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int m = (int)(i / N), n = (int)(i % N);
        float s = 0.f;
        for (int z = 0; z < splits; ++z) s += partial[((size_t)z * M + m) * N + n];
        const int row = idx ? idx[m] : m;
        if (OUT_F32) reinterpret_cast<float *>(Y)[(size_t)row * N + n] = s;
        else reinterpret_cast<__nv_bfloat16 *>(Y)[(size_t)row * N + n] = __float2bfloat16_rn(s);
    }
}

// Routed batches: copy the listed rows of X into a dense [Mcap][K] buffer; slots past the count
// are zero-filled so that the tensor core never sees uninitialised memory.
__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint16_t *__restrict__ X, int K, int Mcap, const int32_t *__restrict__ idx,
                   const int32_t *__restrict__ count, int coff, uint16_t *__restrict__ Xg) {
    pdl_wait();  // the row list comes from the kernel before this one
    pdl_launch_dependents();
    const int rows = min(*count - coff, Mcap);
    const int vec_per_row = K / 8;
    const size_t total = (size_t)Mcap * vec_per_row;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int slot = (int)(i / vec_per_row), v = (int)(i % vec_per_row);
        uint4 val = make_uint4(0, 0, 0, 0);
        if (slot < rows) val = *reinterpret_cast<const uint4 *>(X + (size_t)idx[slot] * K + v * 8);
        *reinterpret_cast<uint4 *>(Xg + (size_t)slot * K + v * 8) = val;
    }
}

template <int MODE, int BN>
dmr_status_t launch_gemm_t(const CUtensorMap &map_w, const CUtensorMap &map_x, const GemmArgs &a, int splits,
                           dmr_out_t out, cudaStream_t st) {
    using Cfg = GemmCfg<MODE, BN>;
    dim3 grid((a.N + BM - 1) / BM, (a.M + BN - 1) / BN, splits);
    auto launch = [&](auto kernel) -> dmr_status_t {
        if (!ensure_dynamic_smem(reinterpret_cast<const void *>(kernel), Cfg::SMEM)) return DMR_ERR_CUDA;
        cudaError_t e = launch_pdl(kernel, grid, dim3(Cfg::THREADS), Cfg::SMEM, st, map_w, map_x, a);
        if (e != cudaSuccess) {
            g_last_cuda_error = (int)e;
            (void)cudaGetLastError();
            return DMR_ERR_CUDA;
        }
        return check_launch();
    };
    if (out == DMR_OUT_F32) return launch(gemm_kernel<MODE, BN, true>);
    return launch(gemm_kernel<MODE, BN, false>);
}

template <int MODE>
dmr_status_t launch_gemm_bn(int BN, const CUtensorMap &map_w, const CUtensorMap &map_x, const GemmArgs &a, int splits,
                            dmr_out_t out, cudaStream_t st) {
    switch (BN) {
        case 32: return launch_gemm_t<MODE, 32>(map_w, map_x, a, splits, out, st);
        case 64: return launch_gemm_t<MODE, 64>(map_w, map_x, a, splits, out, st);
        case 256:
            if constexpr (MODE == 0) return launch_gemm_t<MODE, 256>(map_w, map_x, a, splits, out, st);
        default: return launch_gemm_t<MODE, 128>(map_w, map_x, a, splits, out, st);
    }
}

}  // namespace

bool gemm_supported(int M, int N, int K, int bits /*0 = dense*/, int g) {
    (void)N;
    if (M <= 16 || K % BK != 0) return false;
    if (bits != 0 && bits != 4 && bits != 8) return false;
    if (bits != 0 && (g % BK != 0)) return false;
    return true;
}

GemmPlan gemm_plan(int M, int N, int K, int bits) {
    GemmPlan p;
    p.bn = M <= 32 ? 32 : (M <= 64 ? 64 : 128);
    if (bits == 0 && M > 128) p.bn = 256;
    const int tiles = ((N + BM - 1) / BM) * ((M + p.bn - 1) / p.bn);
    const int kb = K / BK;
    // Split-K factor: the one with the shortest longest path - waves of CTAs (one CTA per SM at a time) times the k blocks
    // of a split plus a fixed cost per wave; at most 8 splits, at least 8 k blocks each.  (Rounding 148 / tiles up, as an
    // earlier version did, put 160 CTAs on 148 SMs for 40 tiles: a second wave for twelve of them.)
    int splits = 1;
    if (tiles < 148) {
        const int max_splits = kb / 8 > 0 ? (kb / 8 < 8 ? kb / 8 : 8) : 1;
        long long best = -1;
        for (int sp = 1; sp <= max_splits; ++sp) {
            const long long waves = ((long long)tiles * sp + 147) / 148;
            const long long cost = waves * ((kb + sp - 1) / sp + 4);
            if (best < 0 || cost < best) {
                best = cost;
                splits = sp;
            }
        }
    }
    p.kblocks_per_split = (kb + splits - 1) / splits;
    p.splits = (kb + p.kblocks_per_split - 1) / p.kblocks_per_split;
    p.partial_bytes = p.splits > 1 ? (size_t)p.splits * M * N * sizeof(float) : 0;
    return p;
}

dmr_status_t launch_gemm(const uint16_t *X, int M, RowSel sel, const void *weights, const uint16_t *scales,
                         const uint8_t *zeros, int N, int K, int bits, int g, void *Y, dmr_out_t out,
                         float *partial, int32_t *status, cudaStream_t st) {
    const GemmPlan p = gemm_plan(M, N, K, bits);
    CUtensorMap map_w, map_x;
    if (!make_tensor_map_2d(&map_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, (uint64_t)M, (uint64_t)K, (uint64_t)K * 2,
                            (uint32_t)p.bn, BK, TmaSwizzle::k128B))
        return DMR_ERR_CUDA;
    if (bits == 0) {
        if (!make_tensor_map_2d(&map_w, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, weights, (uint64_t)N, (uint64_t)K,
                                (uint64_t)K * 2, BM, BK, TmaSwizzle::k128B))
            return DMR_ERR_CUDA;
    } else {
        const uint64_t row_bytes = (uint64_t)K * bits / 8;
        if (!make_tensor_map_2d(&map_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, weights, (uint64_t)N, row_bytes, row_bytes, BM,
                                (uint32_t)(BK * bits / 8), TmaSwizzle::kNone))
            return DMR_ERR_CUDA;
    }
    GemmArgs a;
    a.scales = scales;
    a.zeros = zeros;
    a.Y = Y;
    a.partial = p.splits > 1 ? partial : nullptr;
    a.idx = sel.idx;
    a.count = sel.count;
    a.status = status;
    a.M = M;
    a.N = N;
    a.K = K;
    a.g_size = bits == 0 ? K : g;
    a.kblocks_per_split = p.kblocks_per_split;
    dmr_status_t r;
    if (bits == 0) r = launch_gemm_bn<0>(p.bn, map_w, map_x, a, p.splits, out, st);
    else if (bits == 4) r = launch_gemm_bn<4>(p.bn, map_w, map_x, a, p.splits, out, st);
    else r = launch_gemm_bn<8>(p.bn, map_w, map_x, a, p.splits, out, st);
    if (r != DMR_OK) return r;
    if (p.splits > 1) r = launch_splitk_reduce(partial, p.splits, M, N, sel, Y, out, st);
    return r;
}

dmr_status_t launch_splitk_reduce(const float *partial, int splits, int M, int N, RowSel sel, void *Y, dmr_out_t out,
                                  cudaStream_t st) {
    const size_t total = (size_t)M * N / ((N & 3) == 0 ? 4 : 1);
    int blocks = (int)((total + 255) / 256);
    if (blocks > 148 * 8) blocks = 148 * 8;
    if (out == DMR_OUT_F32)
        (void)launch_pdl(splitk_reduce_kernel<true>, dim3((unsigned)blocks), dim3(256), 0, st, partial, splits, M, N, sel.idx, sel.count, Y);
    else
        (void)launch_pdl(splitk_reduce_kernel<false>, dim3((unsigned)blocks), dim3(256), 0, st, partial, splits, M, N, sel.idx, sel.count, Y);
    return check_launch();
}

dmr_status_t launch_gather_rows(const uint16_t *X, int K, int Mcap, const int32_t *idx, const int32_t *count,
                                int coff, uint16_t *Xg, cudaStream_t st) {
    const size_t total = (size_t)Mcap * (K / 8);
    int blocks = (int)((total + 255) / 256);
    if (blocks > 148 * 8) blocks = 148 * 8;
    (void)launch_pdl(gather_rows_kernel, dim3((unsigned)blocks), dim3(256), 0, st, X, K, Mcap, idx, count, coff, Xg);
    return check_launch();
}

}  // namespace dmr
