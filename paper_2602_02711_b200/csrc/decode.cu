// Decode-time linear layers (M <= 16 rows): bandwidth-bound kernels that stream the weight
// matrix exactly once.  Decoding re-streams the model weights for every generated token and is
// limited by memory bandwidth, which is where weight-only quantization pays (App. "Evaluation
// protocol", discussion of output length; App. "Latency coefficients").
//
// Shape of the computation.  A CTA owns 16*R consecutive output features and its 8 warps split K
// into 8 contiguous slices; partial sums meet in shared memory and are added in warp order, so
// the summation order of an output depends on (K) only - not on M, on the row's position in the
// batch or on the other rows.  Inside a warp the product runs on the tensor cores with the
// weights as the 16-row operand of mma.m16n8k16 (bf16 in, fp32 accumulate) and up to 8 (or
// 2 x 8) activation rows as the 8-column operand.
//
// Low-bit weights: every warp runs its own TMA pipeline (cp.async.bulk.tensor into a private ring
// of 128-byte-swizzled [16R rows x 128 bytes] boxes, one mbarrier per stage), so many kilobytes
// per SM are in flight without costing registers.  Codes are unpacked with one LOP3 per two codes
// ((w >> 4p) & 0x000F000F | 0x43004300 = {128+q_p, 128+q_{p+4}} as two bf16) and one packed
// subtract of (128 + zero): the tensor-core operand is the exact integer q - zero.  Products are
// accumulated per quantization group in fp32 and the group's scale is applied to the group sum,
// so no weight is ever rounded: the only error against exact arithmetic is fp32 summation.
// Which k each fragment slot holds is free as long as both operands agree, so the activation
// fragments are permuted to the unpack order instead of the weights; which feature each fragment
// row holds is free too, which is used to make the shared-memory reads conflict-free.
#include <cuda_bf16.h>

#include "sm100.cuh"

namespace dmr {

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;

__device__ __forceinline__ uint4 ldg_stream(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ uint4 ldg_cached(const void *p) {
    return __ldg(reinterpret_cast<const uint4 *>(p));
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t lop3_and_or(uint32_t a, uint32_t mask, uint32_t orv) {
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(a), "r"(mask), "r"(orv));  // (a & b) | c
    return r;
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}

__device__ __forceinline__ uint32_t bf16x2_sub(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

__device__ __forceinline__ uint32_t bf16x2_mul(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

__device__ __forceinline__ uint32_t pack_bf16x2_rn(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Row of X (and of Y) that batch slot `slot` stands for; -1 if the slot is empty.
__device__ __forceinline__ int slot_row(int slot, int rows, const int32_t *idx) {
    if (slot >= rows) return -1;
    return idx ? idx[slot] : slot;
}

// Fragment row g of a 16-row tile holds tile row tile_row_of(g) (and that + 8).
template <int BITS>
__device__ __forceinline__ int tile_row_of(int g) {
    // 4-bit: rows 0,4,1,5,... so that the eight lanes of one shared-memory phase (two values of g)
    // land on different 16-byte columns under the 128-byte swizzle.  Otherwise identity.
    return BITS == 4 ? ((g >> 1) | ((g & 1) << 2)) : g;
}

// Cross-warp reduction in fixed warp order and store of the CTA's [16R features] x [8NT slots].
// Warp w parks its partial sums at red + w * WSTRIDE floats.
template <int BITS, int NT, int R, int WSTRIDE, bool OUT_F32>
__device__ __forceinline__ void reduce_and_store(float (&acc)[R][NT][4], float *red, int n0, int N,
                                                 int rows, const int32_t *idx, void *Y) {
    constexpr int FEAT = 16 * R, SLOTS = 8 * NT;
    static_assert(WSTRIDE >= FEAT * SLOTS, "partial-sum area too small");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int trow = tile_row_of<BITS>(g);
    float *mine = red + (size_t)warp * WSTRIDE;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int s0 = nt * 8 + 2 * t;
            mine[(s0 + 0) * FEAT + r * 16 + trow] = acc[r][nt][0];
            mine[(s0 + 1) * FEAT + r * 16 + trow] = acc[r][nt][1];
            mine[(s0 + 0) * FEAT + r * 16 + trow + 8] = acc[r][nt][2];
            mine[(s0 + 1) * FEAT + r * 16 + trow + 8] = acc[r][nt][3];
        }
    __syncthreads();
    for (int o = threadIdx.x; o < FEAT * SLOTS; o += kThreads) {
        const int slot = o / FEAT, f = o % FEAT;
        const int row = slot_row(slot, rows, idx);
        const int n = n0 + f;
        if (row < 0 || n >= N) continue;
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) s += red[(size_t)w * WSTRIDE + o];
        if (OUT_F32)
            reinterpret_cast<float *>(Y)[(size_t)row * N + n] = s;
        else
            reinterpret_cast<__nv_bfloat16 *>(Y)[(size_t)row * N + n] = __float2bfloat16_rn(s);
    }
}

// ---------------------------------------------------------------------------------------------
// Low-bit weights.  One step of a warp = one TMA box = 128 bytes of each of 16R feature rows
// (256 4-bit codes or 128 8-bit codes).  A step is consumed in units of UNIT = 128 or 64
// consecutive k (one quantization group, or a part of one); in a unit, lane (g = lane/4,
// t = lane%4) owns codes [t*UNIT/4, (t+1)*UNIT/4) of two feature rows per 16-row tile.
// ---------------------------------------------------------------------------------------------
template <int BITS, int NT, int R, int UNIT, int D, bool OUT_F32>
__global__ void __launch_bounds__(kThreads, 1)
decode_lowbit_kernel(const __grid_constant__ CUtensorMap wmap, const uint16_t *__restrict__ X, int M,
                     const int32_t *__restrict__ idx, const int32_t *__restrict__ count, int coff,
                     const uint16_t *__restrict__ scales, const uint8_t *__restrict__ zeros, int N, int K,
                     int g_size, void *__restrict__ Y, int32_t *__restrict__ status) {
    constexpr int STEP_K = 128 * 8 / BITS;       // codes per 128-byte row
    constexpr int UNITS = STEP_K / UNIT;         // units per step
    constexpr int CPL = UNIT / 4;                // codes per lane per unit
    constexpr int BPL = CPL * BITS / 8;          // bytes per lane per unit (8, 16 or 32)
    constexpr int WPL = BPL / 4;                 // 32-bit words per lane per unit
    constexpr int XV = CPL / 8;                  // 16-byte activation loads per lane per unit
    constexpr int ROWS = 16 * R;
    constexpr int STAGE_BYTES = ROWS * 128;
    extern __shared__ __align__(1024) uint8_t smem_raw[];

    const int rows = count ? min(*count - coff, M) : M;
    if (rows <= 0) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int n0 = blockIdx.x * ROWS;
    const int G = K / g_size;

    uint8_t *my_stages = smem_raw + (size_t)warp * D * STAGE_BYTES;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_raw + (size_t)kWarps * D * STAGE_BYTES) + warp * D;
    const uint32_t stage0 = smem_u32(my_stages);
    const uint32_t bar0 = smem_u32(bars);

    const int steps = (K + STEP_K - 1) / STEP_K;
    const int spw = (steps + kWarps - 1) / kWarps;
    const int s_begin = warp * spw;
    const int my_steps = max(0, min(steps, s_begin + spw) - s_begin);

    if (lane == 0) {
        for (int d = 0; d < D; ++d) mbar_init(bar0 + 8 * d, 1);
        fence_barrier_init();
        for (int d = 0; d < D && d < my_steps; ++d) {
            mbar_expect_tx(bar0 + 8 * d, STAGE_BYTES);
            tma_load_2d(stage0 + d * STAGE_BYTES, &wmap, bar0 + 8 * d, (s_begin + d) * 128, n0);
        }
    }
    __syncwarp();

    // tile rows / features of this lane, activation rows of this lane's fragment column
    const int trow = tile_row_of<BITS>(g);
    int feat[R][2];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        feat[r][0] = min(n0 + r * 16 + trow, N - 1);
        feat[r][1] = min(n0 + r * 16 + trow + 8, N - 1);
    }
    int xrow[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) xrow[nt] = slot_row(nt * 8 + g, rows, idx);

    float acc[R][NT][4], accg[R][NT][4];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[r][nt][c] = accg[r][nt][c] = 0.f;

    // byte offset of this lane inside a 128-byte row for unit u, before swizzling
    const uint32_t lane_row_off[2] = {(uint32_t)(trow * 128), (uint32_t)((trow + 8) * 128)};
    const uint32_t swz = (uint32_t)(trow & 7);  // (trow + 8) & 7 is the same

    bool ok = true;
    for (int i = 0; i < my_steps && ok; ++i) {
        const int d = i % D;
        ok = mbar_wait(bar0 + 8 * d, (uint32_t)((i / D) & 1), status);
        if (!ok) break;
        const uint32_t st = stage0 + d * STAGE_BYTES;
        const int kstep = (s_begin + i) * STEP_K;
#pragma unroll
        for (int u = 0; u < UNITS; ++u) {
            const int k0 = kstep + u * UNIT;
            if (k0 >= K) break;  // warp-uniform: the box reached past the end of the row
            const int grp = k0 / g_size;

            // activations: the two bf16 at k = kc + 2j, kc + 2j + 1 in xb[nt][j]
            const int kc = k0 + t * CPL;
            uint32_t xb[NT][4 * XV];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                if (xrow[nt] >= 0) {
                    const uint16_t *xp = X + (size_t)xrow[nt] * K + kc;
#pragma unroll
                    for (int v = 0; v < XV; ++v) {
                        uint4 q = ldg_cached(xp + 8 * v);
                        xb[nt][4 * v + 0] = q.x;
                        xb[nt][4 * v + 1] = q.y;
                        xb[nt][4 * v + 2] = q.z;
                        xb[nt][4 * v + 3] = q.w;
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 4 * XV; ++j) xb[nt][j] = 0u;
                }
            }
            // zero points of (feature, group)
            uint32_t zb[R][2];
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int h = 0; h < 2; ++h) zb[r][h] = __ldg(zeros + (size_t)feat[r][h] * G + grp);

            const uint32_t boff = (uint32_t)(u * (UNIT * BITS / 8) + t * BPL);  // logical byte in the row
#pragma unroll
            for (int r = 0; r < R; ++r) {
                // packed codes of this lane: rows trow and trow + 8 of tile r
                uint32_t wq[2][WPL];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t rowbase = st + r * 2048 + lane_row_off[h];
#pragma unroll
                    for (int c = 0; c < (BPL + 15) / 16; ++c) {
                        const uint32_t chunk = ((boff >> 4) + c) ^ swz;
                        const uint32_t addr = rowbase + (chunk << 4) + (boff & 15u);
                        if (BPL >= 16) {
                            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                         : "=r"(wq[h][4 * c + 0]), "=r"(wq[h][4 * c + 1]), "=r"(wq[h][4 * c + 2]),
                                           "=r"(wq[h][4 * c + 3])
                                         : "r"(addr));
                        } else {
                            asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(wq[h][0]), "=r"(wq[h][1]) : "r"(addr));
                        }
                    }
                }
                if (BITS == 4) {
                    uint32_t zoff[2];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint32_t zz = 0x4300u | zb[r][h];  // bf16 of 128 + zero (exact)
                        zoff[h] = zz | (zz << 16);
                    }
#pragma unroll
                    for (int w = 0; w < WPL; ++w) {
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            uint32_t a[4];
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                const uint32_t uu = wq[h][w];
                                const uint32_t v0 = lop3_and_or(uu >> (8 * hh), 0x000F000Fu, 0x43004300u);
                                const uint32_t v1 = lop3_and_or(uu >> (8 * hh + 4), 0x000F000Fu, 0x43004300u);
                                a[h] = bf16x2_sub(v0, zoff[h]);      // codes p, p+4 (p = 2hh) minus zero
                                a[2 + h] = bf16x2_sub(v1, zoff[h]);  // codes p+1, p+5
                            }
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt) {
                                // activations in the same order: (x_p, x_{p+4}) and (x_{p+1}, x_{p+5})
                                const uint32_t r0 = xb[nt][4 * w + hh], r2 = xb[nt][4 * w + 2 + hh];
                                mma_bf16_16816(accg[r][nt], a[0], a[1], a[2], a[3], prmt(r0, r2, 0x5410),
                                               prmt(r0, r2, 0x7632));
                            }
                        }
                    }
                } else {
                    float zf[2];
#pragma unroll
                    for (int h = 0; h < 2; ++h) zf[h] = __uint_as_float(0x4B000000u | zb[r][h]);  // 2^23 + zero
#pragma unroll
                    for (int w = 0; w < WPL; ++w) {
                        uint32_t a[4];
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const uint32_t uu = wq[h][w];
                            float f[4];
#pragma unroll
                            for (int b = 0; b < 4; ++b)  // (2^23 + byte) - (2^23 + zero) = q - zero exactly
                                f[b] = __fsub_rn(__uint_as_float(prmt(uu, 0x4B000000u, 0x7650u + (uint32_t)b)), zf[h]);
                            a[h] = pack_bf16x2_rn(f[0], f[1]);  // |q - zero| <= 255: exact in bf16
                            a[2 + h] = pack_bf16x2_rn(f[2], f[3]);
                        }
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt)
                            mma_bf16_16816(accg[r][nt], a[0], a[1], a[2], a[3], xb[nt][2 * w], xb[nt][2 * w + 1]);
                    }
                }
            }
            // end of a quantization group (or of this warp's slice): apply the group's scale
            const bool last_unit = (i == my_steps - 1) && (u == UNITS - 1 || k0 + UNIT >= K);
            if (((k0 + UNIT) % g_size) == 0 || last_unit) {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const float s0 = __uint_as_float((uint32_t)__ldg(scales + (size_t)feat[r][0] * G + grp) << 16);
                    const float s1 = __uint_as_float((uint32_t)__ldg(scales + (size_t)feat[r][1] * G + grp) << 16);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        acc[r][nt][0] = fmaf(s0, accg[r][nt][0], acc[r][nt][0]);
                        acc[r][nt][1] = fmaf(s0, accg[r][nt][1], acc[r][nt][1]);
                        acc[r][nt][2] = fmaf(s1, accg[r][nt][2], acc[r][nt][2]);
                        acc[r][nt][3] = fmaf(s1, accg[r][nt][3], acc[r][nt][3]);
#pragma unroll
                        for (int c = 0; c < 4; ++c) accg[r][nt][c] = 0.f;
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0 && i + D < my_steps) {
            mbar_expect_tx(bar0 + 8 * d, STAGE_BYTES);
            tma_load_2d(st, &wmap, bar0 + 8 * d, (s_begin + i + D) * 128, n0);
        }
    }
    // (a wait that ran out has already lasted far longer than any copy takes: nothing is in flight)
    __syncwarp();
    // this warp's partial sums go to the start of its own (now idle) stage memory
    float *red = reinterpret_cast<float *>(smem_raw);
    reduce_and_store<BITS, NT, R, D * STAGE_BYTES / 4, OUT_F32>(acc, red, n0, N, rows, idx, Y);
}

// ---------------------------------------------------------------------------------------------
// bf16 weights (the high-precision rows).  One step = 64 consecutive k; lane (g, t) owns
// k = 32i + 8t .. +8 (i = 0, 1) of the step for features g and g+8.
// ---------------------------------------------------------------------------------------------
template <int NT, int R, bool OUT_F32>
__global__ void __launch_bounds__(kThreads, 1)
decode_dense_kernel(const uint16_t *__restrict__ X, int M, const int32_t *__restrict__ idx,
                    const int32_t *__restrict__ count, int coff, const uint16_t *__restrict__ W, int N, int K,
                    void *__restrict__ Y) {
    extern __shared__ float red[];
    const int rows = count ? min(*count - coff, M) : M;
    if (rows <= 0) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int n0 = blockIdx.x * 16 * R;

    const int steps = K / 64;
    const int spw = (steps + kWarps - 1) / kWarps;
    const int s_begin = warp * spw, s_end = min(steps, s_begin + spw);

    int frow[R][2];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        frow[r][0] = min(n0 + r * 16 + g, N - 1);
        frow[r][1] = min(n0 + r * 16 + g + 8, N - 1);
    }
    int xrow[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) xrow[nt] = slot_row(nt * 8 + g, rows, idx);

    float acc[R][NT][4];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[r][nt][c] = 0.f;

    uint4 wv[R][2][2];
    auto load_weights = [&](int s) {
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int i = 0; i < 2; ++i)
                    wv[r][h][i] = ldg_stream(W + (size_t)frow[r][h] * K + (size_t)s * 64 + 32 * i + 8 * t);
    };
    if (s_begin < s_end) load_weights(s_begin);

    for (int s = s_begin; s < s_end; ++s) {
        uint4 xv[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                if (xrow[nt] >= 0)
                    xv[nt][i] = ldg_cached(X + (size_t)xrow[nt] * K + (size_t)s * 64 + 32 * i + 8 * t);
                else
                    xv[nt][i] = make_uint4(0, 0, 0, 0);
            }
        uint4 cur[R][2][2];
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int i = 0; i < 2; ++i) cur[r][h][i] = wv[r][h][i];
        if (s + 1 < s_end) load_weights(s + 1);
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int i = 0; i < 2; ++i)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    mma_bf16_16816(acc[r][nt], cur[r][0][i].x, cur[r][1][i].x, cur[r][0][i].y,
                                   cur[r][1][i].y, xv[nt][i].x, xv[nt][i].y);
                    mma_bf16_16816(acc[r][nt], cur[r][0][i].z, cur[r][1][i].z, cur[r][0][i].w,
                                   cur[r][1][i].w, xv[nt][i].z, xv[nt][i].w);
                }
    }
    reduce_and_store<0, NT, R, 16 * R * 8 * NT, OUT_F32>(acc, red, n0, N, rows, idx, Y);
}

// ---------------------------------------------------------------------------------------------
// Any-shape fallback: one warp per output feature, fp32 FMAs, lanes stride over k in chunks of 8.
// ---------------------------------------------------------------------------------------------
template <int MODE /*0 dense, 4, 8*/, bool OUT_F32>
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
                if (MODE == 4) {
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

// Features per CTA: keep at least ~2 CTAs per SM when N allows it.
int pick_r(int N) {
    if (N >= 148 * 2 * 64) return 4;
    if (N >= 148 * 2 * 32) return 2;
    return 1;
}

template <typename KernelT>
dmr_status_t set_smem(KernelT kernel, size_t bytes) {
    if (bytes > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
        if (e != cudaSuccess) {
            g_last_cuda_error = (int)e;
            return DMR_ERR_CUDA;
        }
    }
    return DMR_OK;
}

template <int R>
constexpr int stages_for() { return R == 1 ? 4 : (R == 2 ? 3 : 2); }

template <int BITS, int NT, int R, int UNIT>
dmr_status_t launch_lowbit_t(const uint16_t *X, int M, RowSel sel, const uint32_t *qweight,
                             const uint16_t *scales, const uint8_t *zeros, int N, int K, int g, void *Y,
                             dmr_out_t out, int32_t *status, cudaStream_t st) {
    constexpr int D = stages_for<R>();
    constexpr int ROWS = 16 * R;
    const size_t smem = (size_t)kWarps * D * ROWS * 128 + (size_t)kWarps * D * 8;
    const int grid = (N + ROWS - 1) / ROWS;
    CUtensorMap wmap;
    const uint64_t row_bytes = (uint64_t)K * BITS / 8;
    if (!make_tensor_map_2d(&wmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, qweight, (uint64_t)N, row_bytes, row_bytes, ROWS,
                            128, TmaSwizzle::k128B))
        return DMR_ERR_CUDA;
    if (out == DMR_OUT_F32) {
        auto k = decode_lowbit_kernel<BITS, NT, R, UNIT, D, true>;
        if (set_smem(k, smem) != DMR_OK) return DMR_ERR_CUDA;
        k<<<grid, kThreads, smem, st>>>(wmap, X, M, sel.idx, sel.count, sel.offset, scales, zeros, N, K, g, Y, status);
    } else {
        auto k = decode_lowbit_kernel<BITS, NT, R, UNIT, D, false>;
        if (set_smem(k, smem) != DMR_OK) return DMR_ERR_CUDA;
        k<<<grid, kThreads, smem, st>>>(wmap, X, M, sel.idx, sel.count, sel.offset, scales, zeros, N, K, g, Y, status);
    }
    return check_launch();
}

template <int BITS, int NT, int UNIT>
dmr_status_t launch_lowbit_r(int R, const uint16_t *X, int M, RowSel sel, const uint32_t *qweight,
                             const uint16_t *scales, const uint8_t *zeros, int N, int K, int g, void *Y,
                             dmr_out_t out, int32_t *status, cudaStream_t st) {
    switch (R) {
        case 4: return launch_lowbit_t<BITS, NT, 4, UNIT>(X, M, sel, qweight, scales, zeros, N, K, g, Y, out, status, st);
        case 2: return launch_lowbit_t<BITS, NT, 2, UNIT>(X, M, sel, qweight, scales, zeros, N, K, g, Y, out, status, st);
        default: return launch_lowbit_t<BITS, NT, 1, UNIT>(X, M, sel, qweight, scales, zeros, N, K, g, Y, out, status, st);
    }
}

template <int BITS, int UNIT>
dmr_status_t launch_lowbit_nt(int R, const uint16_t *X, int M, RowSel sel, const uint32_t *qweight,
                              const uint16_t *scales, const uint8_t *zeros, int N, int K, int g, void *Y,
                              dmr_out_t out, int32_t *status, cudaStream_t st) {
    if (M <= 8) return launch_lowbit_r<BITS, 1, UNIT>(R, X, M, sel, qweight, scales, zeros, N, K, g, Y, out, status, st);
    return launch_lowbit_r<BITS, 2, UNIT>(R > 2 ? 2 : R, X, M, sel, qweight, scales, zeros, N, K, g, Y, out, status, st);
}

template <int NT, int R>
dmr_status_t launch_dense_t(const uint16_t *X, int M, RowSel sel, const uint16_t *W, int N, int K, void *Y,
                            dmr_out_t out, cudaStream_t st) {
    const size_t smem = (size_t)kWarps * 16 * R * 8 * NT * sizeof(float);
    const int grid = (N + 16 * R - 1) / (16 * R);
    if (out == DMR_OUT_F32) {
        auto k = decode_dense_kernel<NT, R, true>;
        if (set_smem(k, smem) != DMR_OK) return DMR_ERR_CUDA;
        k<<<grid, kThreads, smem, st>>>(X, M, sel.idx, sel.count, sel.offset, W, N, K, Y);
    } else {
        auto k = decode_dense_kernel<NT, R, false>;
        if (set_smem(k, smem) != DMR_OK) return DMR_ERR_CUDA;
        k<<<grid, kThreads, smem, st>>>(X, M, sel.idx, sel.count, sel.offset, W, N, K, Y);
    }
    return check_launch();
}

}  // namespace

// The unit of k a warp consumes at a time: a whole 128-wide group (or a 128-wide part of a longer
// one), else 64.
static int unit_for(int g) { return g % 128 == 0 ? 128 : (g % 64 == 0 ? 64 : 0); }

bool decode_lowbit_supported(int M, int N, int K, int bits, int g) {
    (void)N;
    const int unit = unit_for(g);
    return M >= 1 && M <= 16 && unit != 0 && K % unit == 0 && (bits == 4 || bits == 8);
}

dmr_status_t launch_decode_lowbit(const uint16_t *X, int M, RowSel sel, const uint32_t *qweight,
                                  const uint16_t *scales, const uint8_t *zeros, int N, int K, int bits,
                                  int g, void *Y, dmr_out_t out, int32_t *status, cudaStream_t st) {
    const int R = pick_r(N);
    const int unit = unit_for(g);
    if (bits == 4) {
        if (unit == 128) return launch_lowbit_nt<4, 128>(R, X, M, sel, qweight, scales, zeros, N, K, g, Y, out, status, st);
        return launch_lowbit_nt<4, 64>(R, X, M, sel, qweight, scales, zeros, N, K, g, Y, out, status, st);
    }
    if (unit == 128) return launch_lowbit_nt<8, 128>(R, X, M, sel, qweight, scales, zeros, N, K, g, Y, out, status, st);
    return launch_lowbit_nt<8, 64>(R, X, M, sel, qweight, scales, zeros, N, K, g, Y, out, status, st);
}

bool decode_dense_supported(int M, int N, int K) {
    (void)N;
    return M >= 1 && M <= 16 && K % 64 == 0;
}

dmr_status_t launch_decode_dense(const uint16_t *X, int M, RowSel sel, const uint16_t *W, int N, int K,
                                 void *Y, dmr_out_t out, cudaStream_t st) {
    const int R = pick_r(N) >= 2 ? 2 : 1;
    if (M <= 8) {
        if (R == 2) return launch_dense_t<1, 2>(X, M, sel, W, N, K, Y, out, st);
        return launch_dense_t<1, 1>(X, M, sel, W, N, K, Y, out, st);
    }
    if (R == 2) return launch_dense_t<2, 2>(X, M, sel, W, N, K, Y, out, st);
    return launch_dense_t<2, 1>(X, M, sel, W, N, K, Y, out, st);
}

dmr_status_t launch_simple_lowbit(const uint16_t *X, int M, RowSel sel, const uint32_t *qweight,
                                  const uint16_t *scales, const uint8_t *zeros, int N, int K, int bits,
                                  int g, void *Y, dmr_out_t out, cudaStream_t st) {
    const int grid = (N + 7) / 8;
    if (bits == 4) {
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
