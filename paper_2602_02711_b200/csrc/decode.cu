// Decode-time 4-bit (and 3-bit) linear layer (up to 16 rows per launch): the weight matrix is read exactly once.
// Decoding re-streams the model weights for every generated token and is limited by memory
// bandwidth, which is where weight-only quantization pays (App. "Evaluation protocol", discussion of output
// length; App. "Latency coefficients").
//
// Work decomposition.  The output features are cut into tiles of 16 R rows; CTA c of a grid of one CTA per SM
// owns a contiguous range of tiles and, for each of them, the whole k range, so no sum ever crosses a CTA:
// there is no scratch memory, no counter and no wait on another CTA in this kernel.  Inside the CTA all warps
// work on the same tile and split its k range in boxes of 256 input features (box b goes to warp b % WARPS).
// The partial sums of every output are added in warp order through shared memory - a fixed order that depends
// on the instance and the layer's shape only, so a row's result never depends on the batch around it.  The hand-over
// is by mbarrier: a warp announces its sums of a tile and adds up the tile before, so the loop has no CTA-wide barrier.
//
// Data movement.  Every warp has a ring of its own in shared memory that one of its lanes keeps full with TMA
// boxes of [16 R rows x 128 bytes] of packed codes (two or four chunks; rows past N read as zero; 128-byte
// swizzle; 3-bit codes: rows of 96 bytes, not swizzled); nobody else reads it, so the only synchronisation is
// the warp's own mbarrier per stage.  The boxes
// are as large as the tile allows because every box costs the SM's copy engine a fixed time of its own
// (measured: about 70 cycles, whatever its size).  A tile's scales and zero points are two contiguous blocks
// of the tables; one thread copies them to shared memory three tiles ahead (bulk copies) when the layer's shape
// allows it, otherwise they are read from global memory where they are needed.  Activations come through the
// L1 with ordinary loads issued a chunk's worth of arithmetic ahead, piece by piece as their registers fall free.
//
// Inner loop.  Lane (g, t) (g = lane / 4, t = lane % 4) takes WPL consecutive code words of two rows of each
// 16-row block and the 8 WPL activations they meet for batch rows g (and g + 8 in the 16-row instance).
// ((w >> 4p) & 0x000F000F) | 0x43004300 is the bf16 pair {128 + q_p, 128 + q_{p+4}} - exact - and goes to the
// tensor cores as it is (mma.m16n8k16, the weights as the 16-row operand), a byte permute pairs the
// activations the same way, and MMAs with an all-ones operand give the sum of the chunk's activations per batch
// row (the common layer shapes form these sums in the CTA's first tile only and keep them in shared memory: they do
// not depend on the tile).  3-bit codes: 32 codes in three words, five per half-word - (w >> 3i) & 0x00070007 is the
// pair of codes i and i + 5 of a word, the pair at bits 3..5 is taken unshifted as 128 + 8 q and brought to 128 + q by
// one bf16 fma.  A chunk never crosses a quantization group, so per chunk
//     sum_k x_k s (q_k - z) = s (sum_k x_k (128 + q_k) - (128 + z) sum_k x_k)
// is formed in fp32 from the two accumulators: no weight is rounded, the zero point costs nothing per weight,
// and the error against exact arithmetic is fp32 summation of terms about thirty times the result (a few
// 1e-7 of the largest output, measured).
//
// Launch chains.  The kernel lets its successor start at once (programmatic dependent launch) and asks for
// more than half of an SM's shared memory, so that an SM never holds two CTAs of these kernels: the
// successor's CTA moves in when this kernel's CTA on that SM has finished, fills its rings and only then waits
// for its predecessor.  (Bulk prefetches of the CTA's whole share into the L2 were tried on top of the rings and
// cost more issue slots than they saved: 159 against 147 us per sweep of twelve layers.)  (With two CTAs per SM
// the successor's CTAs land wherever a slot happens to be free - two on
// some SMs, none on others - and the kernel runs at the pace of the doubly loaded SMs; measured with in-kernel
// time stamps.)  Weights, scales and zero points are read before the wait: they must not be produced by a
// kernel that releases its dependents early (the library's own kernels that write weights never do).
#include <cuda_bf16.h>

#include <cstdlib>

#include "sm100.cuh"

namespace dmr {

namespace {


struct DecodeArgs {
    const uint16_t *X;        // [*][K] bf16
    const int32_t *idx;       // routed: row of X / Y for batch slot s (nullptr = identity)
    const int32_t *count;     // routed: valid slots in the whole list (nullptr = M)
    const uint32_t *qweight;  // [N][K bits / 32]
    const uint16_t *scales;   // [N][G] bf16
    const uint8_t *zeros;     // [N][G]
    void *Y;                  // [*][N]
    int32_t *status;          // set to DMR_ERR_TIMEOUT if a bounded wait runs out
    int M, coff, N, K, G;
    int g_shift;              // log2(group size) when it is a power of two, else -1
    int g_size;
    int tiles;                // ceil(N / tile rows)
    int nchunks;              // K / chunk size
    int sz_stage;             // 1: a tile's scales and zero points are copied to shared memory ahead of time
    int sz_vec;               // 1: the entries of a box's groups are consecutive, aligned and read with one load each (shared or global)
    int sz_zoff, sz_stride;   // shared-memory offset of a tile's zero points; bytes between the tile buffers
    int sx_off, sx_warp;      // FAST: shared-memory offset of the cached activation sums; bytes per warp
};

__device__ __forceinline__ uint4 ldg_v4(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
// Copies `bytes` (a multiple of 16, both addresses 16-byte aligned) from global to shared memory; completes on `bar`.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src),
                 "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds_v2(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts_f32x2(uint32_t addr, float x, float y) {
    asm volatile("st.shared.v2.f32 [%0], {%1,%2};" ::"r"(addr), "f"(x), "f"(y) : "memory");
}
__device__ __forceinline__ float2 lds_f32x2(uint32_t addr) {
    float2 v;
    asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t addr) {
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds_u8(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

constexpr size_t kMinSmem = 116 * 1024;  // more than half of the 228 KB of an SM
constexpr int kSzBuffers = 3;  // tiles whose scales and zero points are in shared memory at a time

template <int BITS, int NT, int R, int WPL, int WARPS, int D>
struct DecodeCfg {
    static_assert(BITS == 4 || (BITS == 3 && WPL == 4), "3-bit codes come in blocks of 32: chunks of 128 input features");
    static constexpr int THREADS = WARPS * 32;
    static constexpr int TILE = 16 * R;
    static constexpr int CHUNK_K = 32 * WPL;
    static constexpr int CHUNK_BYTES = CHUNK_K * BITS / 8;
    static constexpr int BOX_BYTES = BITS == 3 ? 96 : 128;    // bytes of a row in one TMA box (4 bits: the 128-byte swizzle span)
    static constexpr int CPB = BOX_BYTES / CHUNK_BYTES;       // chunks per box
    static constexpr int STAGE_BYTES = TILE * BOX_BYTES;
    static constexpr int NACC = R * NT * 4;
    static constexpr int RING_BYTES = WARPS * D * STAGE_BYTES;
    static constexpr int RED_BUFS = 2;                         // tile t's sums are written while tile t - 1's are added up
    static constexpr int RED_BYTES = RED_BUFS * WARPS * NACC * 32 * 4;
    static constexpr int BAR_OFF = RING_BYTES + RED_BYTES;     // WARPS * D ring barriers, kSzBuffers table barriers, RED_BUFS sum barriers
    static constexpr int SZ_OFF = BAR_OFF + ((WARPS * D + kSzBuffers + RED_BUFS) * 8 + 15) / 16 * 16;
    static constexpr size_t SMEM = (size_t)SZ_OFF + 1024 /*alignment slack*/;  // plus kSzBuffers * sz_stride when staging
};

// NT: 8-row activation blocks (1 or 2).  R: 16-row weight blocks per tile.  WPL: code words per lane and
// row in one chunk (4: chunks of 128 input features, for groups that are multiples of 128; 2: chunks of
// 64, for groups of 64).  WARPS: warps per CTA.  D: stages of a warp's ring.
// FAST: the common layer shape, fixed at compile time so that the hot loop carries no shape tests - every tile is
// whole and its scales and zero points are staged in shared memory, a chunk is one quantization group, K is a whole
// number of boxes, and the sums of the activations per chunk (which do not depend on the tile) fit in shared memory:
// they are formed during the CTA's first tile and read back afterwards.
template <int BITS, int NT, int R, int WPL, int WARPS, int D, bool OUT_F32, bool FAST>
__global__ void __launch_bounds__(WARPS * 32, 1) decode_w4_kernel(const __grid_constant__ CUtensorMap wmap, const DecodeArgs a) {
    using Cfg = DecodeCfg<BITS, NT, R, WPL, WARPS, D>;
    constexpr int TILE = Cfg::TILE, CHUNK_K = Cfg::CHUNK_K, NACC = Cfg::NACC, THREADS = Cfg::THREADS, CPB = Cfg::CPB;
    extern __shared__ uint8_t smem_dyn[];
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    float *red = reinterpret_cast<float *>(smem_dyn + (base - smem_u32(smem_dyn)) + Cfg::RING_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    // box row of fragment row g: 0, 4, 1, 5, ... for 4-bit codes (bank-conflict-free under the swizzle); 3-bit boxes are not swizzled
    const int pg = BITS == 3 ? g : ((g >> 1) | ((g & 1) << 2));
    // 4-bit codes: where this lane's words of fragment row g and chunk 0 sit inside a stage
    const uint32_t lane_off = (uint32_t)(pg * Cfg::BOX_BYTES) + (WPL == 4 ? (uint32_t)((t ^ pg) << 4) : (uint32_t)((((t >> 1) ^ pg) << 4) + (t & 1) * 8));
    const int t0 = (int)(((long long)blockIdx.x * a.tiles) / gridDim.x);
    const int t1 = (int)(((long long)(blockIdx.x + 1) * a.tiles) / gridDim.x);
    const uint32_t ring = base + (uint32_t)warp * (D * Cfg::STAGE_BYTES);
    const uint32_t bars = base + Cfg::BAR_OFF + (uint32_t)warp * (D * 8);
    const uint32_t szbars = base + Cfg::BAR_OFF + WARPS * D * 8;
    const uint32_t redbars = szbars + kSzBuffers * 8;  // "every warp has written its sums of this tile", one per buffer
    const uint32_t szbuf = base + Cfg::SZ_OFF;
    const uint32_t sxbase = base + (uint32_t)a.sx_off + (uint32_t)(warp * a.sx_warp);  // FAST: this warp's cached activation sums
    const int nboxes = (a.nchunks + CPB - 1) / CPB;

    // Every warp sets up its own ring and starts its first copies at once; the barriers of the shared scale / zero-point
    // buffers are warp 0's, and the one CTA-wide barrier that makes them visible comes after the copies are under way.
    if (threadIdx.x == 0) prefetch_tensor_map(&wmap);
    if (lane == 0) {
#pragma unroll
        for (int d = 0; d < D; ++d) mbar_init(bars + 8 * d, 1);
        if (warp == 0) {
#pragma unroll
            for (int d = 0; d < kSzBuffers; ++d) mbar_init(szbars + 8 * d, 1);
#pragma unroll
            for (int d = 0; d < Cfg::RED_BUFS; ++d) mbar_init(redbars + 8 * d, WARPS);
        }
        fence_barrier_init();
    }
    __syncwarp();
    pdl_launch_dependents();

    // ---- a tile's scales and zero points into shared memory (two contiguous blocks of the tables) ----
    int sz_issued = 0;
    auto issue_sz = [&](int tile) {  // by thread 0; tiles in the order this CTA takes them
        if (!(FAST || a.sz_stage) || tile >= t1) return;
        const int d = sz_issued % kSzBuffers;
        const uint32_t n_entries = (uint32_t)(TILE * a.G);  // staging is only chosen when every tile is whole
        mbar_expect_tx(szbars + 8 * d, n_entries * 3);
        bulk_copy_g2s(szbuf + d * a.sz_stride, a.scales + (size_t)tile * n_entries, n_entries * 2, szbars + 8 * d);
        bulk_copy_g2s(szbuf + d * a.sz_stride + a.sz_zoff, a.zeros + (size_t)tile * n_entries, n_entries, szbars + 8 * d);
        ++sz_issued;
    };
    // ---- this warp's list of steps: tiles t0, t0 + 1, ...; boxes warp, warp + WARPS, ... of each ----
    const bool has_boxes = warp < nboxes;
    bool ok = true;  // false once a bounded wait ran out: the warp stops copying, waiting and storing but still meets every barrier
    int i_tile = t0, i_box = warp, issued = 0;  // the next box to request
    auto issue = [&]() {
        if (!has_boxes || i_tile >= t1 || !ok) return;
        if (lane == 0) {
            const int d = issued % D;
            mbar_expect_tx(bars + 8 * d, Cfg::STAGE_BYTES);
            tma_load_2d(ring + d * Cfg::STAGE_BYTES, &wmap, bars + 8 * d, i_box * Cfg::BOX_BYTES, i_tile * TILE);
        }
        ++issued;
        i_box += WARPS;
        if (i_box >= nboxes) {
            i_box = warp;
            ++i_tile;
        }
    };
#pragma unroll
    for (int d = 0; d < D; ++d) issue();
    if (threadIdx.x == 0) {
#pragma unroll
        for (int d = 0; d < kSzBuffers; ++d) issue_sz(t0 + d);
    }
    __syncthreads();  // warp 0's barriers are set up before anyone waits on them

    pdl_wait();
    const int rows = a.count ? min(*a.count - a.coff, a.M) : a.M;
    if (rows <= 0 || t1 <= t0) {
        // nothing to do (a routed call without rows of this kind): let the copies already under way land first
        for (int d = 0; d < D && d < issued; ++d) mbar_wait(bars + 8 * d, 0u, a.status);
        if (threadIdx.x == 0)
            for (int d = 0; d < sz_issued; ++d) mbar_wait(szbars + 8 * d, 0u, a.status);
        return;
    }

    // this lane's activation rows (batch slot nt * 8 + g; slots past the batch read the first row again: their
    // columns of the products are never stored)
    const uint16_t *xrow[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int slot = nt * 8 + g < rows ? nt * 8 + g : 0;
        xrow[nt] = a.X + (size_t)(a.idx ? a.idx[slot] : slot) * a.K + t * (8 * WPL);
    }
    uint32_t x[NT][WPL][4];  // 8 activations per code word of the chunk to come
    auto load_x = [&](int chunk) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int j = 0; j < WPL; ++j) {
                const uint4 v = ldg_v4(xrow[nt] + chunk * CHUNK_K + 8 * j);
                x[nt][j][0] = v.x;
                x[nt][j][1] = v.y;
                x[nt][j][2] = v.z;
                x[nt][j][3] = v.w;
            }
    };
    if (has_boxes) load_x(warp * CPB);
    // B fragments: the chunk's activations paired like the codes.  4-bit word j: (x0, x4), (x1, x5), (x2, x6), (x3, x7);
    // 3-bit block: pair p = 5 j + i is (x[10 j + i], x[10 j + i + 5]), pair 15 is (x30, x31).
    auto xfrag4 = [&](int nt, int j, int q) -> uint32_t {
        return prmt(x[nt][j][q >> 1], x[nt][j][(q >> 1) + 2], (q & 1) ? 0x7632u : 0x5410u);
    };
    auto xfrag3 = [&](int nt, int p) -> uint32_t {
        if (p == 15) return x[nt][3][3];
        const int lo = 10 * (p / 5) + p % 5, hi = lo + 5;  // activations 2 v, 2 v + 1 are in word v
        return prmt(x[nt][lo >> 3][(lo >> 1) & 3], x[nt][hi >> 3][(hi >> 1) & 3], ((hi & 1) ? 0x7600u : 0x5400u) | ((lo & 1) ? 0x32u : 0x10u));
    };

    float acc[R][NT][4];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[r][nt][c] = 0.f;

    // Adds the warps' sums of tile `tile` (the CTA's tile number `tl`) in warp order and writes the outputs.
    auto finish_tile = [&](int tile, int tl) {
        if (ok) ok = mbar_wait(redbars + 8 * (tl & 1), (uint32_t)((tl >> 1) & 1), a.status);
        // every warp is past that tile's table: its buffer takes the tile kSzBuffers further on
        if (threadIdx.x == 0 && ok) issue_sz(tile + kSzBuffers);
        const float *rbuf = red + (size_t)(tl & 1) * WARPS * (NACC * 32);
        for (int o = threadIdx.x; o < NACC * 32; o += THREADS) {
            const int e = o >> 5, l = o & 31;
            const int c = e & 3, nt = (e >> 2) % NT, r = (e >> 2) / NT;
            const int slot = nt * 8 + 2 * (l & 3) + (c & 1);
            if (slot >= rows) continue;  // a batch column nobody asked for
            float v = rbuf[e * 32 + l];
#pragma unroll
            for (int w2 = 1; w2 < WARPS; ++w2) v += rbuf[(w2 * NACC + e) * 32 + l];
            const int lg = l >> 2;
            const int n = tile * TILE + r * 16 + (BITS == 3 ? lg : ((lg >> 1) | ((lg & 1) << 2))) + 8 * (c >> 1);
            if (ok && n < a.N) {
                const int row = a.idx ? a.idx[slot] : slot;
                if (OUT_F32) reinterpret_cast<float *>(a.Y)[(size_t)row * a.N + n] = v;
                else reinterpret_cast<__nv_bfloat16 *>(a.Y)[(size_t)row * a.N + n] = __float2bfloat16_rn(v);
            }
        }
    };

    int consumed = 0;
    constexpr uint32_t kOnes = 0x3F803F80u;  // bf16 1.0 twice
    for (int tile = t0, tl = 0; tile < t1; ++tile, ++tl) {
        // where the lane's rows' scales and zero points are: element offsets into the tables (global or the tile's copy)
        uint32_t szo[R][2];
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int n = min(tile * TILE + pg + r * 16 + h * 8, a.N - 1);
                szo[r][h] = (uint32_t)((FAST || a.sz_stage) ? n - tile * TILE : n) * (uint32_t)a.G;
            }
        const uint32_t sbase = szbuf + (uint32_t)(tl % kSzBuffers) * a.sz_stride, zbase = sbase + a.sz_zoff;
        if ((FAST || a.sz_stage) && ok) ok = mbar_wait(szbars + 8 * (tl % kSzBuffers), (uint32_t)((tl / kSzBuffers) & 1), a.status);
        const bool form_sx = !FAST || tl == 0;  // FAST: the activation sums are formed in the first tile and kept
        for (int box = warp, bl = 0; box < nboxes; box += WARPS, ++bl) {
            const int d = consumed % D;
            if (ok) ok = mbar_wait(bars + 8 * d, (uint32_t)((consumed / D) & 1), a.status);
            ++consumed;
            const uint32_t stage = ring + d * Cfg::STAGE_BYTES;
            const int nsub = FAST ? CPB : min(CPB, a.nchunks - box * CPB);
            const int grp0 = FAST ? box * CPB  // a chunk is a group
                                  : (a.g_shift >= 0 ? ((box * CPB * CHUNK_K) >> a.g_shift) : ((box * CPB * CHUNK_K) / a.g_size));
            // scales and zero points of the box's groups when they sit side by side in the tile's copy
            uint32_t scv[R][2][CPB / 2], zpv[R][2];
            if (FAST || a.sz_vec) {
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint32_t o = szo[r][h] + (uint32_t)grp0;
                        if (FAST || a.sz_stage) {
                            if constexpr (CPB == 2) {
                                scv[r][h][0] = lds_u32(sbase + 2 * o);
                                zpv[r][h] = lds_u16(zbase + o);
                            } else {
                                const uint2 v = lds_v2(sbase + 2 * o);
                                scv[r][h][0] = v.x;
                                scv[r][h][CPB / 2 - 1] = v.y;
                                zpv[r][h] = lds_u32(zbase + o);
                            }
                        } else {  // tables too large to stage: the same aligned loads from global memory
                            if constexpr (CPB == 2) {
                                scv[r][h][0] = __ldg(reinterpret_cast<const uint32_t *>(a.scales + o));
                                zpv[r][h] = __ldg(reinterpret_cast<const uint16_t *>(a.zeros + o));
                            } else {
                                const uint2 v = __ldg(reinterpret_cast<const uint2 *>(a.scales + o));
                                scv[r][h][0] = v.x;
                                scv[r][h][CPB / 2 - 1] = v.y;
                                zpv[r][h] = __ldg(reinterpret_cast<const uint32_t *>(a.zeros + o));
                            }
                        }
                    }
            }
#pragma unroll
            for (int sub = 0; sub < CPB; ++sub) {
                if (!FAST && sub >= nsub) break;
                const int chunk = box * CPB + sub;
                // scale and 128 + zero point (both as fp32 bits) of this chunk's group for the lane's rows
                uint32_t sc[R][2], zp[R][2];
                if (FAST || a.sz_vec) {
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const uint32_t pair = scv[r][h][sub / 2];
                            sc[r][h] = (sub & 1) ? (pair & 0xFFFF0000u) : (pair << 16);
                            zp[r][h] = prmt(zpv[r][h], 0x00004300u, 0x5044u | ((uint32_t)sub << 8));  // fp32 bits of 128 + z
                        }
                } else {
                    const int k0 = chunk * CHUNK_K;
                    const uint32_t grp = (uint32_t)(a.g_shift >= 0 ? (k0 >> a.g_shift) : (k0 / a.g_size));
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            if (a.sz_stage) {
                                sc[r][h] = lds_u16(sbase + 2 * (szo[r][h] + grp)) << 16;
                                zp[r][h] = (lds_u8(zbase + szo[r][h] + grp) | 0x4300u) << 16;
                            } else {
                                sc[r][h] = (uint32_t)__ldg(a.scales + szo[r][h] + grp) << 16;
                                zp[r][h] = ((uint32_t)__ldg(a.zeros + szo[r][h] + grp) | 0x4300u) << 16;
                            }
                        }
                }
                // the chunk whose activations are fetched during this one (after the CTA's last chunk the warp's first
                // chunk once more: always a valid address)
                const int next_chunk = sub == nsub - 1 ? (box + WARPS < nboxes ? box + WARPS : warp) * CPB : chunk + 1;
                float gs[R][NT][4], sx[NT][4];
                const uint32_t sxaddr = sxbase + (uint32_t)(((bl * CPB + sub) * NT) * 256 + lane * 8);
                if constexpr (FAST) {
                    if (form_sx) {  // the CTA's first tile: an all-ones operand against every B fragment of the chunk
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
                            for (int m = 0; m < 2 * WPL; ++m) {
                                const uint32_t b0 = BITS == 3 ? xfrag3(nt, 2 * m) : xfrag4(nt, m >> 1, 2 * (m & 1));
                                const uint32_t b1 = BITS == 3 ? xfrag3(nt, 2 * m + 1) : xfrag4(nt, m >> 1, 2 * (m & 1) + 1);
                                if (m == 0) mma_bf16_16816_zero(sx[nt], kOnes, kOnes, kOnes, kOnes, b0, b1);
                                else mma_bf16_16816(sx[nt], kOnes, kOnes, kOnes, kOnes, b0, b1);
                            }
                            sts_f32x2(sxaddr + nt * 256, sx[nt][0], sx[nt][1]);
                        }
                    } else {
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            const float2 v = lds_f32x2(sxaddr + nt * 256);
                            sx[nt][0] = sx[nt][2] = v.x;
                            sx[nt][1] = sx[nt][3] = v.y;
                        }
                    }
                }
                if constexpr (BITS == 3) {
                    // Lane (g, t) takes block t of the chunk (32 codes in three words) for rows g and g + 8 of each 16-row
                    // block, and the 32 activations they meet.
                    uint32_t w3[R][2][3];
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const uint32_t addr = stage + (uint32_t)((r * 16 + h * 8 + g) * Cfg::BOX_BYTES + sub * Cfg::CHUNK_BYTES + t * 12);
                            w3[r][h][0] = lds_u32(addr);
                            w3[r][h][1] = lds_u32(addr + 4);
                            w3[r][h][2] = lds_u32(addr + 8);
                        }
                    // Pair p = 5 j + i (j < 3, i < 5) is codes 10 j + i and 10 j + 5 + i of the block - the low and the high
                    // half-word of word j at bit 3 i; pair 15 is codes 30 and 31.  Eight MMAs of two pairs each; the
                    // one with the left-over pair goes first, so that every word of the stage has been used early.
#pragma unroll
                    for (int mi = 0; mi < 8; ++mi) {
                        const int m = (mi + 7) & 7;
                        uint32_t b[NT][2];
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            b[nt][0] = xfrag3(nt, 2 * m);
                            b[nt][1] = xfrag3(nt, 2 * m + 1);
                            if constexpr (!FAST) {
                                if (mi == 0) mma_bf16_16816_zero(sx[nt], kOnes, kOnes, kOnes, kOnes, b[nt][0], b[nt][1]);
                                else mma_bf16_16816(sx[nt], kOnes, kOnes, kOnes, kOnes, b[nt][0], b[nt][1]);
                            }
                        }
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            uint32_t av[4];  // a0..a3: 128 + code, exact in bf16
#pragma unroll
                            for (int q = 0; q < 2; ++q)
#pragma unroll
                                for (int h = 0; h < 2; ++h) {
                                    const int p = 2 * m + q;
                                    uint32_t v;
                                    if (p == 15) {
                                        v = lop3_and_or(w3[r][h][0] >> 15, 0x00010001u, 0x43004300u);
                                        v = lop3_and_or(w3[r][h][1] >> 14, 0x00020002u, v);
                                        v = lop3_and_or(w3[r][h][2] >> 13, 0x00040004u, v);
                                    } else {
                                        const uint32_t u = w3[r][h][p / 5];
                                        const int i = p % 5;
                                        if (i == 0) v = lop3_and_or(u, 0x00070007u, 0x43004300u);
                                        else if (i == 2) v = lop3_and_or(u >> 6, 0x00070007u, 0x43004300u);
                                        else if (i == 4) v = lop3_and_or(u >> 12, 0x00070007u, 0x43004300u);
                                        else  // bits 3..5: 128 + 8 q as it stands; (128 + 8 q) / 8 + 112 = 128 + q on the FMA pipe, exact
                                            v = bf16x2_fma(lop3_and_or(i == 1 ? u : (u >> 6), 0x00380038u, 0x43004300u), 0x3E003E00u, 0x42E042E0u);
                                    }
                                    av[2 * q + h] = v;
                                }
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt) {
                                if (mi == 0) mma_bf16_16816_zero(gs[r][nt], av[0], av[1], av[2], av[3], b[nt][0], b[nt][1]);
                                else mma_bf16_16816(gs[r][nt], av[0], av[1], av[2], av[3], b[nt][0], b[nt][1]);
                            }
                        }
                        if (mi == 0 && sub == nsub - 1) {
                            // every word of the box's last chunk has been used: request the box D ahead into the stage
                            __syncwarp();
                            issue();
                        }
                    }
                } else {
                uint32_t w[R][2][WPL];
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        // this lane's 16 bytes of row pg under the 128-byte swizzle: chunk `sub` flips bits of the
                        // 16-byte column index, the other rows of the fragment are whole kilobytes away
                        const uint32_t rowaddr = ((stage + lane_off) ^ (uint32_t)(sub << (WPL == 4 ? 6 : 5))) + (uint32_t)((r * 16 + h * 8) * Cfg::BOX_BYTES);
                        if constexpr (WPL == 4) {
                            const uint4 v = lds_v4(rowaddr);
                            w[r][h][0] = v.x;
                            w[r][h][1] = v.y;
                            w[r][h][2 % WPL] = v.z;
                            w[r][h][3 % WPL] = v.w;
                        } else {
                            const uint2 v = lds_v2(rowaddr);
                            w[r][h][0] = v.x;
                            w[r][h][1] = v.y;
                        }
                    }
#pragma unroll
                for (int j = 0; j < WPL; ++j) {
                    // activations paired like the codes: (x0, x4), (x1, x5) and (x2, x6), (x3, x7)
                    uint32_t b[NT][4];
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) b[nt][q] = xfrag4(nt, j, q);
                        {   // the registers of this piece are free: fetch the same piece of the chunk to come now, a
                            // chunk's worth of arithmetic ahead of its use (a miss in the L1 costs half a microsecond)
                            const uint4 v = ldg_v4(xrow[nt] + next_chunk * CHUNK_K + 8 * j);
                            x[nt][j][0] = v.x;
                            x[nt][j][1] = v.y;
                            x[nt][j][2] = v.z;
                            x[nt][j][3] = v.w;
                        }
                        if constexpr (!FAST) {
                            if (j == 0) mma_bf16_16816_zero(sx[nt], kOnes, kOnes, kOnes, kOnes, b[nt][0], b[nt][1]);
                            else mma_bf16_16816(sx[nt], kOnes, kOnes, kOnes, kOnes, b[nt][0], b[nt][1]);
                            mma_bf16_16816(sx[nt], kOnes, kOnes, kOnes, kOnes, b[nt][2], b[nt][3]);
                        }
                    }
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        uint32_t av[2][4];  // [pair of MMAs][a0..a3]: 128 + code, exact in bf16
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            // one real shift per word; the shifts by whole bytes are byte permutes, which issue
                            // faster than shifts here (measured: +12 to +20 % on the whole loop)
                            const uint32_t u = w[r][h][j], u4 = u >> 4;
                            av[0][h] = lop3_and_or(u, 0x000F000Fu, 0x43004300u);                          // codes 0, 4
                            av[0][2 + h] = lop3_and_or(u4, 0x000F000Fu, 0x43004300u);                     // codes 1, 5
                            av[1][h] = lop3_and_or(prmt(u, 0u, 0x4321), 0x000F000Fu, 0x43004300u);        // codes 2, 6
                            av[1][2 + h] = lop3_and_or(prmt(u4, 0u, 0x4321), 0x000F000Fu, 0x43004300u);   // codes 3, 7
                        }
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            if (j == 0) mma_bf16_16816_zero(gs[r][nt], av[0][0], av[0][1], av[0][2], av[0][3], b[nt][0], b[nt][1]);
                            else mma_bf16_16816(gs[r][nt], av[0][0], av[0][1], av[0][2], av[0][3], b[nt][0], b[nt][1]);
                            mma_bf16_16816(gs[r][nt], av[1][0], av[1][1], av[1][2], av[1][3], b[nt][2], b[nt][3]);
                        }
                    }
                    if (j == 0 && sub == nsub - 1) {
                        // one word of every shared-memory load of the box's last chunk has been used, so the stage
                        // is in registers: request the box D ahead into it
                        __syncwarp();
                        issue();
                    }
                }
                }  // 4-bit codes
                if constexpr (BITS == 3) load_x(next_chunk);  // (the 4-bit loop fetches piece by piece as it goes)
                // the chunk lies inside one quantization group: s (sum x (128 + q) - (128 + z) sum x)
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const float s0 = __uint_as_float(sc[r][0]), s1 = __uint_as_float(sc[r][1]);
                    const float z0 = __uint_as_float(zp[r][0]), z1 = __uint_as_float(zp[r][1]);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        acc[r][nt][0] = fmaf(s0, fmaf(-z0, sx[nt][0], gs[r][nt][0]), acc[r][nt][0]);
                        acc[r][nt][1] = fmaf(s0, fmaf(-z0, sx[nt][1], gs[r][nt][1]), acc[r][nt][1]);
                        acc[r][nt][2] = fmaf(s1, fmaf(-z1, sx[nt][2], gs[r][nt][2]), acc[r][nt][2]);
                        acc[r][nt][3] = fmaf(s1, fmaf(-z1, sx[nt][3], gs[r][nt][3]), acc[r][nt][3]);
                    }
                }
            }
        }
        // ---- end of a tile.  No CTA-wide barrier: a warp first adds up and writes the outputs of the tile BEFORE (all
        // warps have announced their sums of that one, normally long ago), then puts its own sums of this tile into
        // the other buffer and announces them.  A warp can so run up to one tile ahead of the slowest one, and the
        // buffer it writes is free: whoever announced tile t had finished reading tile t - 1 before.
        if (tl > 0) finish_tile(tile - 1, tl - 1);
        float *rbuf = red + (size_t)(tl & 1) * WARPS * (NACC * 32);
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    rbuf[(warp * NACC + (r * NT + nt) * 4 + c) * 32 + lane] = acc[r][nt][c];
                    acc[r][nt][c] = 0.f;
                }
        __syncwarp();
        if (lane == 0) mbar_arrive(redbars + 8 * (tl & 1));
    }
    finish_tile(t1 - 1, t1 - 1 - t0);
}

int device_sm_count() {
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) cached[dev] = n;
        else cached[dev] = 148;
    }
    return cached[dev];
}

bool decode_pdl_enabled() {
    static int v = -1;
    if (v < 0) {
        const char *e = getenv("DMR_PDL");
        v = (e && e[0] == '0') ? 0 : 1;
    }
    return v != 0;
}

template <int BITS, int NT, int R, int WPL, int WARPS, int D, bool OUT_F32, bool FAST>
dmr_status_t launch_decode_k(const DecodeArgs &a, const CUtensorMap &wmap, int ctas, size_t smem, size_t smem_attr, cudaStream_t st) {
    auto kernel = decode_w4_kernel<BITS, NT, R, WPL, WARPS, D, OUT_F32, FAST>;
    if (!ensure_dynamic_smem(reinterpret_cast<const void *>(kernel), smem_attr)) return DMR_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas, 1, 1);
    cfg.blockDim = dim3(WARPS * 32, 1, 1);
    // more than half of an SM's shared memory: two CTAs of these kernels never share an SM (see above)
    cfg.dynamicSmemBytes = smem < kMinSmem ? kMinSmem : smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    int n_attr = 0;
    if (decode_pdl_enabled()) {
        attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
        ++n_attr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = (unsigned)n_attr;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, wmap, a);
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        (void)cudaGetLastError();
        return DMR_ERR_CUDA;
    }
    return check_launch();
}

template <int BITS, int NT, int R, int WPL, int WARPS, int D, bool OUT_F32>
dmr_status_t launch_decode_t(DecodeArgs a, cudaStream_t st) {
    using Cfg = DecodeCfg<BITS, NT, R, WPL, WARPS, D>;
    constexpr int TILE = Cfg::TILE;
    // shared memory left for the copies of the scale / zero-point tables (227 KB per CTA at most)
    constexpr size_t kSzBudget = 227 * 1024 - Cfg::SMEM < 36 * 1024 ? 227 * 1024 - Cfg::SMEM : 36 * 1024;
    static_assert(Cfg::SMEM <= 227 * 1024, "ring and reduction buffers exceed an SM's shared memory");
    constexpr size_t kSmemMax = 227 * 1024;
    constexpr size_t smem_attr = Cfg::SMEM + kSzBudget < kMinSmem ? kMinSmem : Cfg::SMEM + kSzBudget;
    a.tiles = (a.N + TILE - 1) / TILE;
    a.nchunks = a.K / Cfg::CHUNK_K;
    int ctas = device_sm_count();
    if (ctas > a.tiles) ctas = a.tiles;
    // A tile's scales and zero points are two contiguous blocks of the tables: they are copied to shared memory ahead
    // of time when every tile is whole, the blocks are 16-byte aligned and three tiles' worth stay small.
    const size_t tile_entries = (size_t)TILE * a.G;
    a.sz_zoff = (int)((tile_entries * 2 + 15) / 16 * 16);
    a.sz_stride = a.sz_zoff + (int)((tile_entries + 15) / 16 * 16);
    a.sz_stage = (a.N % TILE == 0 && tile_entries % 16 == 0 && ((uintptr_t)a.scales % 16) == 0 && ((uintptr_t)a.zeros % 16) == 0 &&
                  (size_t)kSzBuffers * a.sz_stride <= kSzBudget) ? 1 : 0;
    // a box covers CPB consecutive groups and every row's entries start at a multiple of CPB
    a.sz_vec = (a.g_size == Cfg::CHUNK_K && a.G % Cfg::CPB == 0 &&
                (a.sz_stage || (((uintptr_t)a.scales % (2 * Cfg::CPB)) == 0 && ((uintptr_t)a.zeros % Cfg::CPB) == 0))) ? 1 : 0;
    size_t smem = Cfg::SMEM + (a.sz_stage ? (size_t)kSzBuffers * a.sz_stride : 0);
    // FAST: the sums of the activations per chunk and batch column, kept from the CTA's first tile on (8 bytes per lane)
    const int nboxes = (a.nchunks + Cfg::CPB - 1) / Cfg::CPB;
    a.sx_off = (int)((smem - 1024 + 15) / 16 * 16);
    a.sx_warp = (nboxes + WARPS - 1) / WARPS * Cfg::CPB * NT * 256;
    const size_t smem_fast = (size_t)a.sx_off + (size_t)WARPS * a.sx_warp + 1024;
    const bool fast = a.sz_stage && a.sz_vec && a.nchunks % Cfg::CPB == 0 && smem_fast <= kSmemMax;
    if (fast) smem = smem_fast;
    CUtensorMap wmap;
    const uint64_t rb = (uint64_t)a.K * BITS / 8;
    if (!make_tensor_map_2d(&wmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a.qweight, (uint64_t)a.N, rb, rb, TILE, Cfg::BOX_BYTES,
                            BITS == 3 ? TmaSwizzle::kNone : TmaSwizzle::k128B))
        return DMR_ERR_CUDA;
    return fast ? launch_decode_k<BITS, NT, R, WPL, WARPS, D, OUT_F32, true>(a, wmap, ctas, smem, kSmemMax, st)
                : launch_decode_k<BITS, NT, R, WPL, WARPS, D, OUT_F32, false>(a, wmap, ctas, smem, smem_attr, st);
}

}  // namespace

bool decode_w4_supported(int M, int N, int K, int g) {
    (void)N;
    if (M < 1 || M > 16) return false;
    if (g == 64) return K % 64 == 0;
    return g % 128 == 0 && K % 128 == 0;
}

// 3-bit codes: blocks of 32 codes never straddle a chunk of 128 input features, and a chunk lies inside one group.
bool decode_w3_supported(int M, int N, int K, int g) {
    (void)N;
    if (M < 1 || M > 16) return false;
    return g % 128 == 0 && K % 128 == 0;
}

// Instances as <NT, R, WPL, WARPS, D>.
#ifndef DMR_DECODE_CFG8
#define DMR_DECODE_CFG8 1, 2, 4, 16, 2
#endif
#ifndef DMR_DECODE_CFG8_G64
#define DMR_DECODE_CFG8_G64 1, 2, 2, 16, 2
#endif
#ifndef DMR_DECODE_CFG16
#define DMR_DECODE_CFG16 2, 2, 4, 8, 2
#endif
#ifndef DMR_DECODE_CFG16_G64
#define DMR_DECODE_CFG16_G64 2, 2, 2, 8, 2
#endif
#ifndef DMR_DECODE3_CFG8
#define DMR_DECODE3_CFG8 1, 2, 4, 16, 2
#endif
#ifndef DMR_DECODE3_CFG16
#define DMR_DECODE3_CFG16 2, 2, 4, 8, 2
#endif

void decode_w4_plan(int M, int g, int *nt, int *r, int *warps) {
    const int cfg8[5] = {DMR_DECODE_CFG8}, cfg8g[5] = {DMR_DECODE_CFG8_G64}, cfg16[5] = {DMR_DECODE_CFG16}, cfg16g[5] = {DMR_DECODE_CFG16_G64};
    const int *c = M <= 8 ? (g == 64 ? cfg8g : cfg8) : (g == 64 ? cfg16g : cfg16);
    *nt = c[0];
    *r = c[1];
    *warps = c[3];
}

void decode_w3_plan(int M, int *nt, int *r, int *warps) {
    const int cfg8[5] = {DMR_DECODE3_CFG8}, cfg16[5] = {DMR_DECODE3_CFG16};
    const int *c = M <= 8 ? cfg8 : cfg16;
    *nt = c[0];
    *r = c[1];
    *warps = c[3];
}

namespace {

DecodeArgs decode_args(const uint16_t *X, int M, RowSel sel, const uint32_t *qweight, const uint16_t *scales, const uint8_t *zeros,
                       int N, int K, int g, void *Y, int32_t *status) {
    DecodeArgs a = {};
    a.X = X;
    a.idx = sel.idx;
    a.count = sel.count;
    a.coff = sel.offset;
    a.qweight = qweight;
    a.scales = scales;
    a.zeros = zeros;
    a.Y = Y;
    a.status = status;
    a.M = M;
    a.N = N;
    a.K = K;
    a.G = K / g;
    a.g_size = g;
    a.g_shift = -1;
    for (int sh = 0; sh < 31; ++sh)
        if ((1 << sh) == g) a.g_shift = sh;
    return a;
}

}  // namespace

dmr_status_t launch_decode_w4(const uint16_t *X, int M, RowSel sel, const uint32_t *qweight, const uint16_t *scales,
                              const uint8_t *zeros, int N, int K, int g, void *Y, dmr_out_t out, int32_t *status,
                              cudaStream_t st, int batch_rows) {
    const DecodeArgs a = decode_args(X, M, sel, qweight, scales, zeros, N, K, g, Y, status);
    const int call_rows = batch_rows > M ? batch_rows : M;
    const bool f32 = out == DMR_OUT_F32;
    if (call_rows <= 8) {
        if (g == 64) return f32 ? launch_decode_t<4, DMR_DECODE_CFG8_G64, true>(a, st) : launch_decode_t<4, DMR_DECODE_CFG8_G64, false>(a, st);
        return f32 ? launch_decode_t<4, DMR_DECODE_CFG8, true>(a, st) : launch_decode_t<4, DMR_DECODE_CFG8, false>(a, st);
    }
    if (g == 64) return f32 ? launch_decode_t<4, DMR_DECODE_CFG16_G64, true>(a, st) : launch_decode_t<4, DMR_DECODE_CFG16_G64, false>(a, st);
    return f32 ? launch_decode_t<4, DMR_DECODE_CFG16, true>(a, st) : launch_decode_t<4, DMR_DECODE_CFG16, false>(a, st);
}

dmr_status_t launch_decode_w3(const uint16_t *X, int M, RowSel sel, const uint32_t *qweight, const uint16_t *scales,
                              const uint8_t *zeros, int N, int K, int g, void *Y, dmr_out_t out, int32_t *status,
                              cudaStream_t st, int batch_rows) {
    const DecodeArgs a = decode_args(X, M, sel, qweight, scales, zeros, N, K, g, Y, status);
    const int call_rows = batch_rows > M ? batch_rows : M;
    const bool f32 = out == DMR_OUT_F32;
    if (call_rows <= 8) return f32 ? launch_decode_t<3, DMR_DECODE3_CFG8, true>(a, st) : launch_decode_t<3, DMR_DECODE3_CFG8, false>(a, st);
    return f32 ? launch_decode_t<3, DMR_DECODE3_CFG16, true>(a, st) : launch_decode_t<3, DMR_DECODE3_CFG16, false>(a, st);
}

}  // namespace dmr
