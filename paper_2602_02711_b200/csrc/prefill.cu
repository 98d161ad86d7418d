// Prefill-sized low-bit linear layers (M in the hundreds and above; 3-, 4- and 8-bit codes): a persistent, warp-specialised
// tcgen05 GEMM with the dequantisation fused into the operand pipeline.  Prefill is a dense
// contraction (its cost is folded into the per-token latency, App. "Latency coefficients"), so it
// belongs on the tensor cores.
//
// Orientation: the weights are the 128-row operand (D[n][m] = sum_k W^[n][k] X[m][k]), one
// tensor-memory lane per output feature, BN (64, 128 or 256) activation rows as the N operand.
//
// Per 64-wide k block and stage of the ring:
//   warp 0      TMA: the packed code tile [128 features x 32 or 64 bytes] and the activation tile
//               [BN rows x 128 bytes, 128-byte swizzle] land in shared memory (one mbarrier);
//   warps 2..9 (2..13 for the 64- and 128-row tiles)  one thread per feature row turns its codes into the fp16 weights s' * (q - zero)
//               (exact integer q - zero, then ONE rounding of the product to 11 significant bits)
//               and stores them as the swizzled K-major A tile;
//   warp 1      one lane issues four tcgen05.mma (128 x BN x 16) that accumulate into one of two
//               fp32 accumulators in tensor memory, and commits the stage back to the producer;
//   the last four warps (eight for the 256-row tile, two per lane quadrant with half of the columns each)
//               drain the finished accumulator of the previous tile (tcgen05.ld) into Y while the
//               next tile's MMAs run into the other accumulator (a block of 32 rows at a time: the rows' scales and
//               output rows come from one coalesced load each, never from loads inside the store loop).
// CTAs are persistent: CTA b takes tiles b, b + grid, ...  Every wait is bounded.
//
// Operand precision.  The MMA runs in fp16 x fp16 -> fp32 (kind::f16) instead of bf16: a bf16 A
// operand would round every dequantized weight to 8 significant bits (1.5e-3 rms relative error of
// the outputs, uncomfortably close to the 2e-3 acceptance bound), fp16 keeps 11 (1.8e-4).  To stay
// inside fp16's range whatever the inputs, a preparation kernel rescales every activation row by a
// power of two (row maximum into [2^13, 2^14): exact for all elements within 2^-27 of the maximum)
// and the unpack threads rescale a feature's scales by the power of two of its largest one; the
// epilogue multiplies the two powers of two back in (exact).
#include <cuda_bf16.h>

#include <type_traits>

#include "sm100.cuh"

namespace dmr {

namespace {

constexpr int PM = 128;  // features per tile (MMA M)
constexpr int PK = 64;   // k per stage

template <int BITS, int BN>
struct PrefillCfg {
    static constexpr int A_BYTES = PM * PK * 2;              // 16 KB of fp16 weights
    static constexpr int B_BYTES = BN * PK * 2;              // activations
    static constexpr int P_ROW = PK * BITS / 8;              // packed bytes per feature per stage
    static constexpr int P_BYTES = BITS == 3 ? 0 : PM * P_ROW;  // 4 or 8 KB (3-bit rows are 24 bytes per stage, which no
                                                                // TMA box can be: the unpack threads read them from global memory)
    static constexpr int STAGE = A_BYTES + B_BYTES + ((P_BYTES + 1023) / 1024) * 1024;
    static constexpr int S_RAW = (212 * 1024) / STAGE;
    static constexpr int S = S_RAW > 8 ? 8 : S_RAW;
    static constexpr int TMEM_COLS = 2 * BN;                 // two accumulators
    // unpack warps: UW / 4 groups of four, group i takes every (UW / 4)-th stage of the ring.  Three groups for the
    // 64- and 128-row tiles (small batches: a stage's MMAs are short and the unpack chain's latency is what is left), two for 256.
    static constexpr int UW = BN == 256 ? 8 : 12;
    // epilogue warps: four (one per tensor-memory lane quadrant), eight for the 256-row tile (two per quadrant, each draining
    // half of the accumulator's columns: what is left after a CTA's last MMA is its last tile's epilogue)
    static constexpr int EW = BN == 256 ? 8 : 4;
    static constexpr int THREADS = 32 * (2 + UW + EW);
    static constexpr size_t SMEM = (size_t)S * STAGE + 1024 /*alignment*/ + 512 /*barriers*/;
};

// Largest magnitude pattern among a feature's G bf16 scales (sign bit cleared): eight scales per 16-byte load when the
// row of the table allows it, so that a work item's set-up is a handful of independent loads, not a chain of G.
__device__ __forceinline__ uint32_t scale_row_max(const uint16_t *sp, int G) {
    uint32_t m0 = 0, m1 = 0;
    int gi = 0;
    // scalar loads up to the first 16-byte boundary, 16-byte loads over the aligned middle, scalar loads for the rest
    const int head = (int)(((16u - (uint32_t)(reinterpret_cast<uintptr_t>(sp) & 15u)) & 15u) >> 1);
    for (; gi < G && gi < head; ++gi) m0 = max(m0, (uint32_t)__ldg(sp + gi) & 0x7FFFu);
    for (; gi + 8 <= G; gi += 8) {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(sp + gi));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            m0 = max(m0, w[i] & 0x7FFFu);
            m1 = max(m1, (w[i] >> 16) & 0x7FFFu);
        }
    }
    for (; gi < G; ++gi) m1 = max(m1, (uint32_t)__ldg(sp + gi) & 0x7FFFu);
    return max(m0, m1);
}

struct PrefillArgs {
    const uint16_t *scales;
    const uint8_t *zeros;
    const uint32_t *qweight3;  // 3-bit codes (read by the unpack threads; 4- and 8-bit codes come through the tensor map)
    const float *xscale;   // power of two each prepared activation row was divided by
    void *Y;
    const int32_t *idx;    // routed: output row of batch slot m (nullptr = identity)
    const int32_t *count;  // routed: number of valid slots (nullptr = M)
    int32_t *status;
    int M, N, K, g_size;
    int n_tiles, m_tiles;
    // split-K (batches of one row tile on layers with few feature tiles): a work item is (tile, split); split z sums the
    // k blocks [z kb_per_split, (z + 1) kb_per_split) and writes fp32 partial sums [z][M][N] that a second kernel adds
    // up in split order.  splits == 1: the tile's whole k range, outputs written directly.
    float *partial;
    int splits, kb_per_split;
};


// Activation preparation: Xh[slot][k] = fp16(X[row(slot)][k] * 2^-e), xscale[slot] = 2^e, with e chosen
// per row so that the row's largest magnitude lands in [2^13, 2^14).  Slots past the valid count
// (routed calls) are zero-filled.  `idx` / `count` as in the GEMM (nullptr = identity).
__device__ __forceinline__ uint32_t row_max_bits(const uint4 &q, uint32_t mx) {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t a0 = w[i] & 0x7FFFu, a1 = (w[i] >> 16) & 0x7FFFu;
        if (a0 < 0x7F80u) mx = max(mx, a0);  // largest FINITE magnitude (bf16 patterns order like magnitudes)
        if (a1 < 0x7F80u) mx = max(mx, a1);
    }
    return mx;
}

__device__ __forceinline__ uint4 to_f16_scaled(const uint4 &q, float down, float down2) {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float f0 = __uint_as_float(w[i] << 16) * down * down2;
        const float f1 = __uint_as_float(w[i] & 0xFFFF0000u) * down * down2;
        asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(o[i]) : "f"(f1), "f"(f0));
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// One CTA of 256 threads per slot (grid-stride over slots); CH = 16-byte chunks a thread keeps in
// registers between the two passes (CH * 256 * 8 >= K), so the row is read from memory once.
template <int CH>
__global__ void __launch_bounds__(256)
xprep_kernel(const uint16_t *__restrict__ X, int K, int Mcap, const int32_t *__restrict__ idx,
             const int32_t *__restrict__ count, uint16_t *__restrict__ Xh, float *__restrict__ xscale) {
    __shared__ uint32_t warp_max[8];
    pdl_wait();               // nothing of the stream's earlier work is read or overwritten before this
    pdl_launch_dependents();  // the GEMM behind this kernel may set itself up meanwhile
    const int rows = count ? min(*count, Mcap) : Mcap;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nv = K / 8;
    for (int slot = blockIdx.x; slot < Mcap; slot += gridDim.x) {
        uint4 *dst = reinterpret_cast<uint4 *>(Xh + (size_t)slot * K);
        if (slot >= rows) {
            for (int v = threadIdx.x; v < nv; v += 256) dst[v] = make_uint4(0, 0, 0, 0);
            if (threadIdx.x == 0) xscale[slot] = 1.f;
            continue;
        }
        const uint4 *src = reinterpret_cast<const uint4 *>(X + (size_t)(idx ? idx[slot] : slot) * K);
        uint4 keep[CH];
        uint32_t mx = 0;
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const int v = c * 256 + threadIdx.x;
            keep[c] = v < nv ? __ldg(src + v) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int c = 0; c < CH; ++c) mx = row_max_bits(keep[c], mx);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
        __syncthreads();  // warp_max of the previous slot has been read by everyone
        if (lane == 0) warp_max[warp] = mx;
        __syncthreads();
#pragma unroll
        for (int w = 0; w < 8; ++w) mx = max(mx, warp_max[w]);
        int eb = (int)(mx >> 7);          // biased exponent of the maximum (0 for zero / subnormal rows)
        if (eb < 1) eb = 1;
        const int e = (eb - 127) - 13;    // x * 2^-e has its maximum in [2^13, 2^14)
        // 2^-e as one or two float factors (|e| can reach 139, beyond one float exponent)
        const float down = e > 0 ? __uint_as_float((uint32_t)(127 - min(e, 126)) << 23) : __uint_as_float((uint32_t)(127 + min(-e, 127)) << 23);
        const float down2 = e < -127 ? __uint_as_float((uint32_t)(127 + (-e - 127)) << 23) : 1.f;
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const int v = c * 256 + threadIdx.x;
            if (v < nv) dst[v] = to_f16_scaled(keep[c], down, down2);
        }
        if (threadIdx.x == 0) xscale[slot] = ldexpf(1.f, e);
    }
}

// SPLITK: work items are (tile, split) and the epilogue writes fp32 partial sums; otherwise an item is a tile with its whole
// k range (a compile-time choice: the large-batch instance carries none of the split bookkeeping).
template <int BITS, int BN, bool OUT_F32, bool SPLITK>
__global__ void __launch_bounds__(PrefillCfg<BITS, BN>::THREADS, 1)
prefill_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, const PrefillArgs a) {
    using Cfg = PrefillCfg<BITS, BN>;
    constexpr int S = Cfg::S;
    extern __shared__ uint8_t smem_dyn[];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
    auto a_tile = [&](int s) { return base + (uint32_t)s * Cfg::STAGE; };
    auto b_tile = [&](int s) { return base + (uint32_t)s * Cfg::STAGE + Cfg::A_BYTES; };
    auto p_tile = [&](int s) { return base + (uint32_t)s * Cfg::STAGE + Cfg::A_BYTES + Cfg::B_BYTES; };
    const uint32_t bar_base = base + (uint32_t)S * Cfg::STAGE;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 64u + 8u * s; };
    auto ready_bar = [&](int s) { return bar_base + 128u + 8u * s; };
    auto tfull_bar = [&](int b) { return bar_base + 192u + 8u * b; };
    auto tempty_bar = [&](int b) { return bar_base + 208u + 8u * b; };
    const uint32_t tmem_slot = bar_base + 224u;
    volatile uint32_t *tmem_slot_ptr = reinterpret_cast<volatile uint32_t *>(base_ptr + S * Cfg::STAGE + 224);

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
            mbar_init(ready_bar(s), 4);   // one arrival per warp of the group that unpacks the stage
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), Cfg::EW);  // one arrival per epilogue warp
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

    // Set-up done (barriers, tensor memory): only now wait for the kernels before this one - the prepared activations, the
    // routed row lists - and let the kernel behind this one (the split-K sum) start its own set-up.
    pdl_wait();
    if constexpr (SPLITK) pdl_launch_dependents();  // (a large batch's successor would only sit on the SMs and wait)
    const int nkb = a.K / PK;
    // a routed call sizes the grid for M rows but only the first `rows` slots hold anything
    const int rows = a.count ? min(*a.count, a.M) : a.M;
    const int n_splits = SPLITK ? a.splits : 1;
    const int total_tiles = a.n_tiles * ((rows + BN - 1) / BN) * n_splits;  // work items: (tile, split), split fastest
    const int G = a.K / a.g_size;
    const int kb_per_group = a.g_size / PK;  // >= 1

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            constexpr uint32_t TX = Cfg::B_BYTES + Cfg::P_BYTES;
            uint32_t it = 0;  // k blocks issued so far, over all tiles
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                const int split = SPLITK ? tile % n_splits : 0, tl = SPLITK ? tile / n_splits : tile;
                const int kb_lo = SPLITK ? split * a.kb_per_split : 0, kb_hi = SPLITK ? min(nkb, kb_lo + a.kb_per_split) : nkb;
                const int n0 = (tl % a.n_tiles) * PM, m0 = (tl / a.n_tiles) * BN;
                for (int kb = kb_lo; kb < kb_hi; ++kb, ++it) {
                    const int s = it % S;
                    if (it >= (uint32_t)S && !mbar_wait(empty_bar(s), ((it / S) - 1) & 1, a.status)) {
                        ok = false;
                        break;
                    }
                    mbar_expect_tx(full_bar(s), TX);
                    tma_load_2d(b_tile(s), &map_x, full_bar(s), kb * PK, m0);
                    if constexpr (BITS != 3) tma_load_2d(p_tile(s), &map_w, full_bar(s), kb * Cfg::P_ROW, n0);
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        // The whole warp runs the loop: stage numbers, descriptors and accumulator addresses are then the same in all
        // lanes (the compiler can keep them in uniform registers, which the MMA instruction reads), and one lane issues.
        {
            constexpr uint32_t IDESC = umma_idesc_f16(PM, BN);
            // Operand descriptors: built once for stage 0; a stage and a k step only move the 14-bit address field (16-byte
            // units), so each MMA costs an add, not a descriptor's worth of dependent shifts and ORs.
            const uint64_t desc_a0 = umma_desc_sw128(a_tile(0)), desc_b0 = umma_desc_sw128(b_tile(0));
            const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
            uint32_t it = 0, tile_it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tile_it) {
                const int buf = tile_it & 1;
                // the epilogue must have drained this accumulator (used two tiles ago)
                if (tile_it >= 2 && !mbar_wait(tempty_bar(buf), ((tile_it >> 1) - 1) & 1, a.status)) break;
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_u + (uint32_t)(buf * BN);
                const int kb_lo = SPLITK ? (tile % n_splits) * a.kb_per_split : 0, kb_hi = SPLITK ? min(nkb, kb_lo + a.kb_per_split) : nkb;
                for (int kb = kb_lo; kb < kb_hi; ++kb, ++it) {
                    const int s = it % S;
                    if (!mbar_wait(ready_bar(s), (it / S) & 1, a.status)) {
                        ok = false;
                        break;
                    }
                    tcgen05_fence_after();
                    const uint64_t stage_off = (uint64_t)(((uint32_t)s * (uint32_t)Cfg::STAGE) >> 4);
                    const uint64_t desc_a = desc_a0 + stage_off, desc_b = desc_b0 + stage_off;
                    if (lane == 0) {
#pragma unroll
                        for (int j = 0; j < PK / 16; ++j)  // 16 k values = 32 bytes of a row = two 16-byte units
                            umma_bf16_ss(d_tmem, desc_a + (uint64_t)(2 * j), desc_b + (uint64_t)(2 * j), IDESC,
                                         (kb == kb_lo && j == 0) ? 0u : 1u);
                        umma_commit(empty_bar(s));
                    }
                    __syncwarp();
                }
                if (ok && lane == 0) umma_commit(tfull_bar(buf));
                __syncwarp();
            }
        }
    } else if (warp < 2 + Cfg::UW) {
        // ================= unpack warps: codes -> fp16 weights s' * (q - zero) =================
        // A stage's chain (wait, load, convert, store, fence, arrive) is a string of shared-memory round trips that
        // one group of four warps cannot overlap with itself, so NG groups work on different stages of the ring
        // at the same time: group i takes the stages whose running number is i modulo NG.
        const int r = ((warp - 2) & 3) * 32 + lane;  // feature row of the tile
        constexpr int NG = Cfg::UW / 4;
        constexpr int CH = 8, c_lo = 0;               // 16-byte chunks (8 weights each) per thread and stage
        const int grp_id = (warp - 2) >> 2;
        const uint32_t swz = (uint32_t)(r & 7);
        uint32_t it0 = 0;  // running number of the work item's first stage
        bool ok = true;
        for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
            const int split = SPLITK ? tile % n_splits : 0, tl = SPLITK ? tile / n_splits : tile;
            const int kb_lo = SPLITK ? split * a.kb_per_split : 0, kb_hi = SPLITK ? min(nkb, kb_lo + a.kb_per_split) : nkb;
            const int n = min((tl % a.n_tiles) * PM + r, a.N - 1);
            const uint16_t *sp = a.scales + (size_t)n * G;
            const uint8_t *zp = a.zeros + (size_t)n * G;
            // power of two of the feature's largest scale: s' = s * 2^-f lies in (0, 2)
            const uint32_t smax = scale_row_max(sp, G);
            int fb = (int)(smax >> 7);
            fb = fb < 1 ? 1 : (fb > 253 ? 253 : fb);
            const float fdown = __uint_as_float((uint32_t)(254 - fb) << 23);  // 2^-(fb - 127)
            int kb = kb_lo + (int)(((uint32_t)grp_id + (uint32_t)NG - it0 % (uint32_t)NG) % (uint32_t)NG);  // this group's first k block of the item
            uint32_t sb = 0, zb = 0;
            if (kb < kb_hi) {
                sb = __ldg(sp + kb / kb_per_group);
                zb = __ldg(zp + kb / kb_per_group);
            }
            // 3-bit codes: this row's six words of the stage, read from global memory one stage of this group ahead
            const uint32_t *wrow = a.qweight3 + (size_t)n * (size_t)(a.K / 32 * 3);
            uint2 w3a = make_uint2(0u, 0u), w3b = w3a, w3c = w3a;
            if (BITS == 3 && kb < kb_hi) {
                w3a = __ldg(reinterpret_cast<const uint2 *>(wrow + kb * 6));
                w3b = __ldg(reinterpret_cast<const uint2 *>(wrow + kb * 6 + 2));
                w3c = __ldg(reinterpret_cast<const uint2 *>(wrow + kb * 6 + 4));
            }
            for (; kb < kb_hi; kb += NG) {
                const uint32_t it = it0 + (uint32_t)(kb - kb_lo);
                const int s = it % S;
                uint2 n3a = w3a, n3b = w3b, n3c = w3c;
                if (BITS == 3 && kb + NG < kb_hi) {
                    n3a = __ldg(reinterpret_cast<const uint2 *>(wrow + (kb + NG) * 6));
                    n3b = __ldg(reinterpret_cast<const uint2 *>(wrow + (kb + NG) * 6 + 2));
                    n3c = __ldg(reinterpret_cast<const uint2 *>(wrow + (kb + NG) * 6 + 4));
                }
                // scale / zero of this group's next k block, fetched while this block is unpacked
                uint32_t sb_next = sb, zb_next = zb;
                if (kb + NG < kb_hi) {
                    const int grp = (kb + NG) / kb_per_group;
                    sb_next = __ldg(sp + grp);
                    zb_next = __ldg(zp + grp);
                }
                if (!mbar_wait(full_bar(s), (it / S) & 1, a.status)) {
                    ok = false;
                    break;
                }
                const uint32_t src = p_tile(s) + r * Cfg::P_ROW;
                const uint32_t dst = a_tile(s) + r * 128;
                if (BITS == 3) {
                    // fp16 patterns: a half-word holds five codes at bits 0, 3, 6, 9, 12.  0x6400 | (bits 0..2) = 1024 + q,
                    // 0x6400 | (bits 3..5) = 1024 + 8 q, 0x6400 | (bits 6..8) = 1024 + 64 q without a shift (10 mantissa
                    // bits); one shift by 9 brings the last two down.  Minus the matching 1024 + zero is exact, then one
                    // rounding of the product with s', s'/8 or s'/64.
                    const float sf = __uint_as_float(sb << 16) * fdown;
                    uint32_t s2, s2_8, s2_64;
                    asm("cvt.rn.f16x2.f32 %0, %1, %1;" : "=r"(s2) : "f"(sf));
                    asm("cvt.rn.f16x2.f32 %0, %1, %1;" : "=r"(s2_8) : "f"(sf * 0.125f));
                    asm("cvt.rn.f16x2.f32 %0, %1, %1;" : "=r"(s2_64) : "f"(sf * 0.015625f));
                    const uint32_t z1 = 0x6400u | zb, z8 = 0x6400u | (zb << 3), z64 = 0x6400u | (zb << 6);
                    const uint32_t zo1 = z1 | (z1 << 16), zo8 = z8 | (z8 << 16), zo64 = z64 | (z64 << 16);
                    const uint32_t words[6] = {w3a.x, w3a.y, w3b.x, w3b.y, w3c.x, w3c.y};
#pragma unroll
                    for (int blk = 0; blk < 2; ++blk) {  // 32 codes = three words = four 16-byte chunks of fp16 weights
                        uint32_t D[16];  // pair 5 j + i = codes (10 j + i, 10 j + 5 + i); pair 15 = codes (30, 31)
#pragma unroll
                        for (int j = 0; j < 3; ++j) {
                            const uint32_t u = words[3 * blk + j], u9 = u >> 9;
                            D[5 * j + 0] = f16x2_mul(f16x2_sub(lop3_and_or(u, 0x00070007u, 0x64006400u), zo1), s2);
                            D[5 * j + 1] = f16x2_mul(f16x2_sub(lop3_and_or(u, 0x00380038u, 0x64006400u), zo8), s2_8);
                            D[5 * j + 2] = f16x2_mul(f16x2_sub(lop3_and_or(u, 0x01C001C0u, 0x64006400u), zo64), s2_64);
                            D[5 * j + 3] = f16x2_mul(f16x2_sub(lop3_and_or(u9, 0x00070007u, 0x64006400u), zo1), s2);
                            D[5 * j + 4] = f16x2_mul(f16x2_sub(lop3_and_or(u9, 0x00380038u, 0x64006400u), zo8), s2_8);
                        }
                        {
                            uint32_t t = lop3_and_or(words[3 * blk] >> 15, 0x00010001u, 0x64006400u);
                            t = lop3_and_or(words[3 * blk + 1] >> 14, 0x00020002u, t);
                            t = lop3_and_or(words[3 * blk + 2] >> 13, 0x00040004u, t);
                            D[15] = f16x2_mul(f16x2_sub(t, zo1), s2);
                        }
                        // code a of the block: pair and half it sits in; the tile wants neighbours (2 v, 2 v + 1) side by side
                        auto pair_of = [](int a) { return a >= 30 ? 15 : 5 * (a / 10) + (a % 10) % 5; };
                        auto high_of = [](int a) { return a >= 30 ? a - 30 : ((a % 10) >= 5 ? 1 : 0); };
#pragma unroll
                        for (int c4 = 0; c4 < 4; ++c4) {
                            uint32_t o[4];
#pragma unroll
                            for (int v4 = 0; v4 < 4; ++v4) {
                                const int a0 = 8 * c4 + 2 * v4, a1 = a0 + 1;
                                o[v4] = prmt(D[pair_of(a0)], D[pair_of(a1)], (high_of(a1) ? 0x7600u : 0x5400u) | (high_of(a0) ? 0x32u : 0x10u));
                            }
                            const uint32_t addr = dst + ((((uint32_t)(4 * blk + c4)) ^ swz) << 4);
                            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
                        }
                    }
                } else if (BITS == 4) {
                    uint32_t w[CH];
#pragma unroll
                    for (int c4 = 0; c4 < CH; c4 += 4)
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                     : "=r"(w[c4]), "=r"(w[c4 + 1]), "=r"(w[c4 + 2]), "=r"(w[c4 + 3])
                                     : "r"(src + 4 * (c_lo + c4)));
                    // fp16 patterns: 0x6400 | q = 1024 + q and 0x6400 | (q << 4) = 1024 + 16 q (no shift needed
                    // for the odd codes); minus 1024 + zero (or 1024 + 16 zero) is exact; then one rounding
                    const float sf = __uint_as_float(sb << 16) * fdown;
                    uint32_t s2, s2_16;
                    asm("cvt.rn.f16x2.f32 %0, %1, %1;" : "=r"(s2) : "f"(sf));
                    asm("cvt.rn.f16x2.f32 %0, %1, %1;" : "=r"(s2_16) : "f"(sf * 0.0625f));
                    const uint32_t zz = 0x6400u | zb, zz16 = 0x6400u | (zb << 4);
                    const uint32_t zoff = zz | (zz << 16), zoff16 = zz16 | (zz16 << 16);
#pragma unroll
                    for (int cc = 0; cc < CH; ++cc) {  // word c = codes 8c .. 8c+7 = 16-byte chunk c of the row
                        const int c = c_lo + cc;
                        const uint32_t w8 = w[cc] >> 8;
                        const uint32_t d04 = f16x2_mul(f16x2_sub(lop3_and_or(w[cc], 0x000F000Fu, 0x64006400u), zoff), s2);
                        const uint32_t d15 = f16x2_mul(f16x2_sub(lop3_and_or(w[cc], 0x00F000F0u, 0x64006400u), zoff16), s2_16);
                        const uint32_t d26 = f16x2_mul(f16x2_sub(lop3_and_or(w8, 0x000F000Fu, 0x64006400u), zoff), s2);
                        const uint32_t d37 = f16x2_mul(f16x2_sub(lop3_and_or(w8, 0x00F000F0u, 0x64006400u), zoff16), s2_16);
                        const uint32_t o01 = prmt(d04, d15, 0x5410), o45 = prmt(d04, d15, 0x7632);
                        const uint32_t o23 = prmt(d26, d37, 0x5410), o67 = prmt(d26, d37, 0x7632);
                        const uint32_t addr = dst + ((((uint32_t)c) ^ swz) << 4);
                        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(o01), "r"(o23), "r"(o45), "r"(o67) : "memory");
                    }
                } else {
                    const float zf = __uint_as_float(0x4B000000u | zb);  // 2^23 + zero
                    const float sf = __uint_as_float(sb << 16) * fdown;
                    // A row of codes is 64 bytes = four 16-byte pieces.  Lane r starts at piece (r / 2) % 4, so that the eight
                    // lanes of a load phase read eight different bank groups (all starting at piece 0 would meet in two).
                    // Piece q holds codes 16 q .. 16 q + 15 = chunks 2 q and 2 q + 1 of the fp16 row.
#pragma unroll
                    for (int j = 0; j < CH / 2; ++j) {
                        const uint32_t q = ((uint32_t)j + (uint32_t)(r >> 1)) & 3u;
                        uint32_t wq[4];
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(wq[0]), "=r"(wq[1]), "=r"(wq[2]), "=r"(wq[3]) : "r"(src + 16u * q));
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            uint32_t o[4];
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                const uint32_t u = wq[2 * e + h];
                                float f[4];
#pragma unroll
                                for (int b = 0; b < 4; ++b)  // (q - zero) exactly, times the scale exactly (8 x 8 bits)
                                    f[b] = __fmul_rn(__fsub_rn(__uint_as_float(prmt(u, 0x4B000000u, 0x7650u + (uint32_t)b)), zf), sf);
                                o[2 * h] = pack_f16x2_rn(f[0], f[1]);  // the one rounding
                                o[2 * h + 1] = pack_f16x2_rn(f[2], f[3]);
                            }
                            const uint32_t addr = dst + (((2u * q + (uint32_t)e) ^ swz) << 4);
                            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
                        }
                    }
                }
                fence_proxy_async_smem();  // the tile must be visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(ready_bar(s));
                sb = sb_next;
                zb = zb_next;
                w3a = n3a;
                w3b = n3b;
                w3c = n3c;
            }
            it0 += (uint32_t)(kb_hi - kb_lo);
        }
    } else {
        // ================= epilogue warps =================
        const int q = warp & 3;        // tensor-memory lane quadrant this warp may read
        constexpr int CW = BN / (Cfg::EW / 4);                   // columns (batch slots) of a tile this warp drains
        const int c_begin = ((warp - 2 - Cfg::UW) >> 2) * CW;
        const int r = q * 32 + lane;   // feature row of the tile
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        uint32_t tile_it = 0;
        for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++tile_it) {
            const int buf = tile_it & 1;
            const int split = SPLITK ? tile % n_splits : 0, tl = SPLITK ? tile / n_splits : tile;
            const int n = (tl % a.n_tiles) * PM + r, m0 = (tl / a.n_tiles) * BN;
            // the power of two the unpack threads divided this feature's scales by, undone here
            const uint32_t smax = scale_row_max(a.scales + (size_t)min(n, a.N - 1) * G, G);
            int fb = (int)(smax >> 7);
            fb = fb < 1 ? 1 : (fb > 253 ? 253 : fb);
            const float fscale = __uint_as_float((uint32_t)fb << 23);  // 2^(fb - 127)
            if (!mbar_wait(tfull_bar(buf), (tile_it >> 1) & 1, a.status)) break;
            tcgen05_fence_after();
#pragma unroll 1
            for (int c0 = c_begin; c0 < c_begin + CW; c0 += 32) {
                uint32_t u[32];
                tmem_ld_x16(lane_addr + (uint32_t)(buf * BN + c0), *reinterpret_cast<uint32_t(*)[16]>(&u[0]));
                tmem_ld_x16(lane_addr + (uint32_t)(buf * BN + c0 + 16), *reinterpret_cast<uint32_t(*)[16]>(&u[16]));
                tmem_ld_wait();
                if (c0 + 32 >= c_begin + CW) {  // this warp's share of the accumulator is in registers: hand it back
                    tcgen05_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tempty_bar(buf));
                }
                // Row scales of this block of 32 batch slots: eight 16-byte loads from one address for the whole warp (the table
                // is padded to a multiple of 64 entries).  A load per element inside the guarded loop below would be a chain of
                // 32 exposed round trips, and every shuffle or load is one more instruction through the memory pipe, which the
                // operand tiles keep busy.  Output rows of a routed call: one coalesced load, handed round by shuffles.
                float xs[32];
                {
                    const float4 *xp = reinterpret_cast<const float4 *>(a.xscale + m0 + c0);
#pragma unroll
                    for (int q4 = 0; q4 < 8; ++q4) {
                        const float4 t = __ldg(xp + q4);
                        xs[4 * q4] = t.x;
                        xs[4 * q4 + 1] = t.y;
                        xs[4 * q4 + 2] = t.z;
                        xs[4 * q4 + 3] = t.w;
                    }
                }
                const bool listed = !SPLITK && a.idx != nullptr;
                const int m_lane = m0 + c0 + lane;
                const int row_lane = (listed && m_lane < rows) ? a.idx[m_lane] : m_lane;
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const int m = m0 + c0 + c;
                    const int row = listed ? __shfl_sync(0xffffffffu, row_lane, c) : m;
                    if (n < a.N && m < rows) {
                        const float v = (__uint_as_float(u[c]) * xs[c]) * fscale;
                        if constexpr (SPLITK) {  // this split's share, by batch slot; the reduction scatters the rows
                            a.partial[((size_t)split * a.M + m) * a.N + n] = v;
                        } else {
                            if (OUT_F32) reinterpret_cast<float *>(a.Y)[(size_t)row * a.N + n] = v;
                            else reinterpret_cast<__nv_bfloat16 *>(a.Y)[(size_t)row * a.N + n] = __float2bfloat16_rn(v);
                        }
                    }
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

template <int BITS, int BN>
dmr_status_t launch_prefill_t(const CUtensorMap &map_w, const CUtensorMap &map_x, const PrefillArgs &a, int grid,
                              dmr_out_t out, cudaStream_t st) {
    using Cfg = PrefillCfg<BITS, BN>;
    auto launch = [&](auto kernel) -> dmr_status_t {
        if (!ensure_dynamic_smem(reinterpret_cast<const void *>(kernel), Cfg::SMEM)) return DMR_ERR_CUDA;
        cudaError_t e = launch_pdl(kernel, dim3((unsigned)grid), dim3(Cfg::THREADS), Cfg::SMEM, st, map_w, map_x, a);
        if (e != cudaSuccess) {
            g_last_cuda_error = (int)e;
            (void)cudaGetLastError();
            return DMR_ERR_CUDA;
        }
        return check_launch();
    };
    if (a.splits > 1) return launch(prefill_kernel<BITS, BN, true, true>);  // partial sums are fp32 whatever the output
    if (out == DMR_OUT_F32) return launch(prefill_kernel<BITS, BN, true, false>);
    return launch(prefill_kernel<BITS, BN, false, false>);
}

int prefill_sm_count() {
    static int cached = 0;
    if (cached == 0) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
            cached = n;
        else
            cached = 148;
    }
    return cached;
}

// Activation rows per tile.  A k block costs a CTA about the same time whatever the tile's width (hand-overs between the
// roles, not MMA time, set the pace), so the wide tile does about twice the work per unit of time; the narrow one is
// for batches it covers alone and for shapes whose last wave it fills much better.  Depends on (M, N) only.
int prefill_bn(int M, int N, int sms) {
    if (M <= 64) return 64;    // one tile of rows: the smaller the activation tile, the more stages are in flight
    if (M <= 128) return 128;
    const int n_tiles = (N + PM - 1) / PM;
    auto score = [&](int bn, double rate) {
        const long long t = (long long)n_tiles * ((M + bn - 1) / bn);
        if (t < sms) return rate;  // fewer tiles than SMs: split along k fills the SMs (prefill_splits)
        const long long waves = (t + sms - 1) / sms;
        return rate * (double)t / (double)(waves * sms);
    };
    return score(256, 1.0) >= score(128, 0.7) ? 256 : 128;  // (measured: the narrow tile wins between 0.67 and 0.75)
}

}  // namespace

bool prefill_supported(int M, int N, int K, int bits, int g) {
    if (!((bits == 3 || bits == 4 || bits == 8) && K % PK == 0 && g % PK == 0 && K <= 32768)) return false;
    if (M > 128 || bits == 3) return M > 32;  // 3-bit codes have no other tensor-core kernel
    // one tile of rows: layers with at least 16 feature tiles (split along k when the tiles alone leave SMs idle); the
    // narrow ones (k and v projections) are faster on the split-K kernel with the exact-integer operand
    return M > 32 && (N + PM - 1) / PM >= 16;
}

// Split-K factor: for shapes whose tiles leave SMs idle.  As many splits as give every SM at most one work item, each
// with at least sixteen k blocks; with more than one row tile the fp32 partial sums are large, and a split is taken only
// if it shortens a work item by at least 48 k blocks.  Depends on (M, N, K) only.
static int prefill_splits(int M, int N, int K, int sms, int *kb_per_split) {
    const int bn = prefill_bn(M, N, sms);
    const int nkb = K / PK, tiles = ((N + PM - 1) / PM) * ((M + bn - 1) / bn);
    int splits = 1;
    if (tiles < sms) {
        splits = sms / tiles;
        if (splits > nkb / 16) splits = nkb / 16;  // a work item pays for its set-up (the feature's scale range) once
        if (splits < 1) splits = 1;
        if (M > 128 && nkb - (nkb + splits - 1) / splits < 48) splits = 1;
    }
    *kb_per_split = (nkb + splits - 1) / splits;
    return (nkb + *kb_per_split - 1) / *kb_per_split;  // no empty split
}

size_t prefill_partial_bytes(int M, int N, int K) {
    int kbps;
    const int splits = prefill_splits(M, N, K, prefill_sm_count(), &kbps);
    return splits > 1 ? (size_t)splits * M * N * sizeof(float) : 0;
}

void prefill_plan(int M, int N, int K, int *bn, int *splits, long long *tiles, int *ctas) {
    const int sms = prefill_sm_count();
    int kbps;
    *bn = prefill_bn(M, N, sms);
    *splits = prefill_splits(M, N, K, sms, &kbps);
    *tiles = (long long)((N + PM - 1) / PM) * ((M + *bn - 1) / *bn);
    const long long items = *tiles * *splits;
    *ctas = (int)(items < sms ? items : sms);
}

size_t prefill_scratch_bytes(int M, int K) { return round_up((size_t)M * K * 2, 256) + round_up((size_t)M * 4, 256); }

dmr_status_t launch_prefill(const uint16_t *X, int M, RowSel sel, const void *qweight, const uint16_t *scales,
                            const uint8_t *zeros, int N, int K, int bits, int g, void *Y, dmr_out_t out,
                            void *scratch, float *partial, int32_t *status, cudaStream_t st) {
    const int sms = prefill_sm_count();
    const int bn = prefill_bn(M, N, sms);
    int kb_per_split;
    const int splits = prefill_splits(M, N, K, sms, &kb_per_split);
    if (splits > 1 && !partial) return DMR_ERR_WORKSPACE;
    // activations: gather (routed calls), rescale each row by a power of two and convert to fp16
    uint16_t *Xh = reinterpret_cast<uint16_t *>(scratch);
    float *xscale = reinterpret_cast<float *>(reinterpret_cast<char *>(scratch) + round_up((size_t)M * K * 2, 256));
    {
        const int blocks = M < sms * 16 ? M : sms * 16;
        cudaError_t e;
        if (K <= 2 * 2048) e = launch_pdl(xprep_kernel<2>, dim3((unsigned)blocks), dim3(256), 0, st, X, K, M, sel.idx, sel.count, Xh, xscale);
        else if (K <= 8 * 2048) e = launch_pdl(xprep_kernel<8>, dim3((unsigned)blocks), dim3(256), 0, st, X, K, M, sel.idx, sel.count, Xh, xscale);
        else if (K <= 16 * 2048) e = launch_pdl(xprep_kernel<16>, dim3((unsigned)blocks), dim3(256), 0, st, X, K, M, sel.idx, sel.count, Xh, xscale);
        else return DMR_ERR_UNSUPPORTED;
        if (e != cudaSuccess) {
            g_last_cuda_error = (int)e;
            (void)cudaGetLastError();
            return DMR_ERR_CUDA;
        }
        dmr_status_t r = check_launch();
        if (r != DMR_OK) return r;
    }
    CUtensorMap map_w, map_x;
    if (!make_tensor_map_2d(&map_x, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, Xh, (uint64_t)M, (uint64_t)K, (uint64_t)K * 2,
                            (uint32_t)bn, PK, TmaSwizzle::k128B))
        return DMR_ERR_CUDA;
    const uint64_t row_bytes = (uint64_t)K * bits / 8;
    if (bits == 3) {
        map_w = map_x;  // not used: a stage of 3-bit codes is 24 bytes per row, the unpack threads load it themselves
    } else if (!make_tensor_map_2d(&map_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, qweight, (uint64_t)N, row_bytes, row_bytes, PM,
                                   (uint32_t)(PK * bits / 8), TmaSwizzle::kNone)) {
        return DMR_ERR_CUDA;
    }
    PrefillArgs a;
    a.scales = scales;
    a.zeros = zeros;
    a.qweight3 = reinterpret_cast<const uint32_t *>(qweight);
    a.xscale = xscale;
    a.Y = Y;
    a.idx = sel.idx;
    a.count = sel.count;
    a.status = status;
    a.M = M;
    a.N = N;
    a.K = K;
    a.g_size = g;
    a.n_tiles = (N + PM - 1) / PM;
    a.m_tiles = (M + bn - 1) / bn;
    a.splits = splits;
    a.kb_per_split = kb_per_split;
    a.partial = splits > 1 ? partial : nullptr;
    const long long tiles = (long long)a.n_tiles * a.m_tiles * splits;
    const int grid = (int)(tiles < sms ? tiles : sms);
    dmr_status_t r;
    auto by_rows = [&](auto bits_tag) -> dmr_status_t {
        constexpr int B = decltype(bits_tag)::value;
        if (bn == 256) return launch_prefill_t<B, 256>(map_w, map_x, a, grid, out, st);
        if (bn == 128) return launch_prefill_t<B, 128>(map_w, map_x, a, grid, out, st);
        return launch_prefill_t<B, 64>(map_w, map_x, a, grid, out, st);
    };
    if (bits == 3) r = by_rows(std::integral_constant<int, 3>{});
    else if (bits == 4) r = by_rows(std::integral_constant<int, 4>{});
    else r = by_rows(std::integral_constant<int, 8>{});
    if (r != DMR_OK || splits == 1) return r;
    return launch_splitk_reduce(partial, splits, M, N, sel, Y, out, st);
}

}  // namespace dmr
