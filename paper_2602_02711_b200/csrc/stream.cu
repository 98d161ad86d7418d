// Decode-time linear layers (up to 32 rows per launch): one persistent kernel that streams the weight matrix
// exactly once at memory speed.  Decoding re-streams the model weights for every generated token
// and is limited by memory bandwidth, which is where weight-only quantization pays (App.
// "Evaluation protocol", discussion of output length; App. "Latency coefficients").
//
// Work decomposition.  The weight matrix is cut into steps of [128 features x 128 bytes] (256
// 4-bit codes, 128 8-bit codes or 64 bf16 weights per feature), numbered feature-group major, k
// minor.  Two ways of dealing the steps out, chosen from the shape alone:
//  - Large layers: CTA c of the persistent grid (one or two CTAs per SM) takes the contiguous range
//    [c * total / ctas, (c + 1) * total / ctas), so every SM streams the same number of bytes whatever
//    the shape.  A feature group whose steps are shared by several CTAs is finished by the last of
//    them to arrive, which adds the partial sums in CTA order.  Counting a CTA into a shared group is
//    a round trip to the L2; one lane of a warp of its own does that while the consumer warps go on
//    with their next steps, and the sums of the groups a CTA was last for are formed at the end of the
//    kernel by all consumer warps.
//  - Small layers (up to 25 MB of codes), where that sum across CTAs is most of the run time:
//    thread-block clusters of eight CTAs (four for the 16- and 32-row kernels).  A cluster owns whole feature
//    groups, rank r streams the r-th part of their k range, and at the end the cluster adds the sums
//    of every output in rank order through distributed shared memory, each CTA taking its share of the
//    outputs.
// Either way there are no floating-point atomics, and the summation order of an output depends on
// (N, K), the device and whether the call has up to 8, up to 16 or more rows - never on the row's
// position in the batch or on the other rows (all chunks of a call use the same kernel instance).
//
// Inside a CTA one producer lane keeps a ring of stages full by TMA (cp.async.bulk.tensor,
// 128-byte swizzle): the weight box and the matching activation boxes, all completing on the
// stage's mbarrier (a routed batch is gathered into consecutive rows beforehand).  Eight consumer
// warps each own 32 features and one half of the step's k range; the product runs on the tensor
// cores with the weights as the 16-row operand of mma.m16n8k16 and 8 activation rows (one, two or
// four such tiles per instance) as the 8-column operand.  4-bit codes are unpacked with one
// LOP3 per two codes ((w >> 4p) & 0x000F000F | 0x43004300 = {128 + q_p, 128 + q_{p+4}} as two
// bf16) and one packed subtract of (128 + zero): the tensor-core operand is the exact integer
// q - zero.  Products are accumulated per quantization group in fp32 and the group's scale is
// applied to the group sum, so no weight is ever rounded: the only error against exact arithmetic
// is fp32 summation.
//
// Programmatic dependent launch: the kernel lets its successor start at once and prefetches its
// own first weight stages before waiting for its predecessor, because weights never depend on
// the previous kernel; activations, row lists and the scratch area are touched only afterwards.
#include <cuda_bf16.h>

#include <cstdlib>

#include "sm100.cuh"

namespace dmr {

namespace {

// Warp geometry.  8 consumer warps of 32 features each, except the 16-row kernel for bf16 weights: it has
// its SM alone and no unpack work to amortise, and runs faster with 16 consumer warps of 16 features
// (measured: +7 %; the 16-row kernels for packed codes lose 6 % that way and keep 8 warps).
__host__ __device__ constexpr int r_tiles(int nt, int bits) { return (nt == 2 && bits == 16) ? 1 : 2; }  // 16-feature tiles per consumer warp
__host__ __device__ constexpr int row_blocks(int nt, int bits) { return 128 / (16 * r_tiles(nt, bits)); }  // consumer warps side by side
__host__ __device__ constexpr int consumer_warps(int nt, int bits) { return 2 * row_blocks(nt, bits); }    // two k halves
__host__ __device__ constexpr int stream_threads(int nt, int bits) { return (consumer_warps(nt, bits) + 2) * 32; }  // + producer + publishing warp
constexpr int kTileRows = 128;                              // features per step
constexpr int kStepBytes = kTileRows * 128;                 // weight bytes per step (16 KB)
constexpr int kMaxStages = 12;
// CTAs that share the k range of a feature group: 8 for the 8-row kernels (two CTAs per SM), 4 for the
// 16-row kernels (one CTA per SM: clusters of 8 SMs would leave a fifth of the SMs without work).
__host__ __device__ constexpr int cluster_size(int nt) { return nt == 1 ? 8 : 4; }
constexpr int kClusterMaxStepsDense = 2100;                // the same for bf16 weights (a 4096 x 4096 layer: 10.7 us instead of 13.9)
constexpr int kClusterMaxSteps = 1600;                     // layers of up to this many steps (25 MB) run in cluster mode
// Shared memory for the stage ring, KB: two 8-row CTAs share an SM, a 16-row CTA has it alone.
__host__ __device__ constexpr int stage_budget_kb(int nt) { return nt == 1 ? 92 : (nt == 2 ? 100 : 136); }






__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}

// Release: the parts this CTA stored (ordered before this lane by the barrier it waited on) are
// visible to whoever reads the new count.  Acquire: if this was the last count, the other CTAs'
// parts are visible to this CTA's loads that follow.
__device__ __forceinline__ int atom_add_acq_rel(int32_t *p, int v) {
    int old;
    asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}

// Fragment row g of a 16-row tile holds tile row tile_row_of(g) (and that + 8): rows 0,4,1,5,...
// so that the eight lanes of one shared-memory phase (two values of g, four 16-byte chunks each)
// land on different bank groups under the 128-byte swizzle.
__device__ __forceinline__ int tile_row_of(int g) { return (g >> 1) | ((g & 1) << 2); }

// Geometry of one step for a weight width.
template <int BITS>
struct StepGeom {
    static constexpr int STEP_K = 1024 / BITS;         // weights per 128-byte row: 256, 128, 64
    static constexpr int UNIT_K = STEP_K / 2;          // per k-half warp: 128, 64, 32
    static constexpr int X_BOXES = STEP_K / 64;        // activation boxes of 64 k (128 bytes per row): 4, 2, 1
};

// Activation boxes of a stage sit (slots * 128 + 256) bytes apart: the box itself plus two rows, so
// that consecutive boxes start two rows further into the 128-byte swizzle pattern (the pattern is tied
// to the shared-memory address, chunk ^= (address / 128) % 8).  Lanes t and t + 2 of a warp read the
// same chunk index of consecutive boxes; the shift sends them to different banks.
__host__ __device__ constexpr int x_box_pitch(int slots) { return slots * 128 + 256; }

// Byte offset, inside a stage's activation area, of 16-byte chunk c (k = 8 c .. 8 c + 7 of the step)
// of batch slot `slot`.
template <int SLOTS>
__device__ __forceinline__ uint32_t x_chunk_offset(int c, int slot) {
    constexpr int PITCH = x_box_pitch(SLOTS);
    const int sb = c >> 3, cc = c & 7;
    return (uint32_t)(sb * PITCH + slot * 128 + ((cc ^ ((slot + 2 * sb) & 7)) << 4));
}

struct StreamArgs {
    const int32_t *idx;       // routed: row of X / Y for batch slot s (nullptr = identity)
    const int32_t *count;     // routed: valid slots in the list (nullptr = M)
    const uint16_t *scales;   // low-bit only
    const uint8_t *zeros;     // low-bit only
    void *Y;
    float *partial;           // [ctas][2][16 slots][128 features] fp32
    int32_t *counters;        // [feature groups][kCounterStride], zero on entry and on exit
    int32_t *status;
    int M, coff, N, K, g_size;
    int g_shift;              // log2(g_size) when it is a power of two, else -1
    int steps_per_group;      // ceil(K / STEP_K)
    int total_steps;          // feature groups * steps_per_group
    int part_groups;          // cluster mode: feature groups whose sums fit into a CTA's shared memory at once
    int tiles;                // host side: 8-row activation tiles of the kernel to launch (1, 2 or 4)
};

__device__ __forceinline__ long long range_begin(int c, int ctas, int total) {
    return ((long long)c * total) / ctas;
}

// ---- thread-block clusters: rank, remote shared-memory addresses, remote barrier arrivals ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_id_x() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_count_x() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r));
    return r;
}
// All threads of all CTAs of the cluster (hardware barrier; used once, after the barriers are set up).
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of this CTA's shared-memory location `addr` in the CTA of rank `rank` of the cluster.
__device__ __forceinline__ uint32_t cluster_map(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Bounded wait that also orders the other CTAs' shared-memory writes before this thread's reads.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, int32_t *status) {
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
        if (i > 128) __nanosleep(64);
    }
    if (status) atomicExch(status, (int32_t)DMR_ERR_TIMEOUT);
    return false;
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t cluster_addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(cluster_addr));
    return v;
}

// Consumer-warp barrier on an mbarrier (one arrival per warp) so that the wait is bounded.
__device__ __forceinline__ bool consumer_sync(uint32_t bar, uint32_t &phase, int32_t *status) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
    const bool ok = mbar_wait(bar, phase, status);
    phase ^= 1u;
    return ok;
}

template <int BITS, int NT, int GS>
struct StreamCfg {
    using G = StepGeom<BITS>;
    static constexpr int SLOTS = NT * 8;
    static constexpr int X_PITCH = x_box_pitch(SLOTS);
    static constexpr int X_STAGE = ((G::X_BOXES * X_PITCH + 1023) / 1024) * 1024;
    static constexpr int X_TX = G::X_BOXES * SLOTS * 128;  // bytes the activation boxes deliver
    static constexpr int STAGE = kStepBytes + X_STAGE;
    static constexpr int D_RAW = (stage_budget_kb(NT) * 1024) / STAGE;
    static constexpr int D = D_RAW > kMaxStages ? kMaxStages : D_RAW;
    static constexpr int SUM_FLOATS = SLOTS * kTileRows;     // the sums k half 1 parks for k half 0
    // cluster mode keeps the sums of several feature groups here until the cluster adds them up
    static constexpr int PART_BYTES = NT == 1 ? (BITS == 16 ? 16 : 20) * 1024 : 64 * 1024;  // 4 to 40 groups at full row count
    static constexpr int PARK_BYTES = 2 * SUM_FLOATS * 4;    // two parking buffers, used in turn
    static constexpr int SCRATCH = PART_BYTES > PARK_BYTES ? PART_BYTES : PARK_BYTES;
    static constexpr int SZ_OFF = D * STAGE + SCRATCH;
    static constexpr int SZ_WARP = 2 * 16 * r_tiles(NT, BITS) * GS * 4;  // per consumer warp: two slots of (scale, zero) entries
    static constexpr int BAR_OFF = SZ_OFF + consumer_warps(NT, BITS) * SZ_WARP;
    static constexpr size_t SMEM = (size_t)BAR_OFF + 512 + 1024 /*alignment slack*/;
};

// BITS: 4 / 8 = packed codes, 16 = bf16 weights.  NT: 8-row activation tiles (1, 2 or 4).
// GS: quantization groups per 128-code unit (2 only for 4-bit codes with 64-wide groups).
// CE: every unit a warp consumes ends its quantization group (group size == unit size).
// CL: the CTAs of a thread-block cluster split the k range of the same feature groups and add their
// sums through distributed shared memory (no trip through the L2); without it, CTAs take contiguous
// step ranges and shared feature groups are summed through global memory by the last to arrive.
template <int BITS, int NT, int GS, bool CE, bool OUT_F32, bool CL>
__global__ void __launch_bounds__(stream_threads(NT, BITS), NT == 1 ? 2 : 1)
decode_stream_kernel(const __grid_constant__ CUtensorMap wmap, const __grid_constant__ CUtensorMap xmap,
                     const StreamArgs a) {
    using Cfg = StreamCfg<BITS, NT, GS>;
    using Geo = StepGeom<BITS>;
    constexpr int D = Cfg::D, SLOTS = Cfg::SLOTS, R = r_tiles(NT, BITS);
    constexpr int kRowBlocks = row_blocks(NT, BITS), kConsumerWarps = consumer_warps(NT, BITS), kPublishWarp = kConsumerWarps + 1;
    constexpr int kClusterSize = cluster_size(NT);
    constexpr int kPartSlots = NT == 4 ? 32 : 16;  // batch slots of a CTA's part of a shared feature group in global memory
    constexpr bool LOWBIT = BITS != 16;
    constexpr int WPS = 4 / GS;  // 32-bit code words per lane, feature and group part
    extern __shared__ uint8_t smem_dyn[];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
    auto w_stage = [&](int d) { return base + (uint32_t)d * kStepBytes; };
    auto x_stage = [&](int d) { return base + (uint32_t)D * kStepBytes + (uint32_t)d * Cfg::X_STAGE; };
    float *scratch = reinterpret_cast<float *>(base_ptr + D * Cfg::STAGE);
    const uint32_t bar0 = base + Cfg::BAR_OFF;
    auto full_bar = [&](int d) { return bar0 + 8u * d; };
    auto empty_bar = [&](int d) { return bar0 + 128u + 8u * d; };
    const uint32_t cons_bar = bar0 + 256u;
    auto pub_bar = [&](int e) { return bar0 + 264u + 8u * e; };    // k half 0 warps -> publishing lane
    auto role_bar = [&](int e) { return bar0 + 280u + 8u * e; };   // publishing lane -> consumer warps
    volatile int32_t *is_last = reinterpret_cast<volatile int32_t *>(base_ptr + Cfg::BAR_OFF + 320);
    const uint32_t cl_full_bar = bar0 + 296u;   // cluster mode: every CTA's sums of the round are in place
    const uint32_t cl_done_bar = bar0 + 304u;   // cluster mode: every CTA has finished reading the others' sums

    const int ctas = gridDim.x, cta = blockIdx.x;
    const int SPG = a.steps_per_group;
    const int G = LOWBIT ? a.K / a.g_size : 1;
    // quantization group of input feature k without a division in the common cases
    auto group_of_k = [&](int k) { return a.g_shift >= 0 ? (k >> a.g_shift) : (G == 1 ? 0 : k / a.g_size); };
    // ---- the work of this CTA ----
    // Without clusters: the contiguous step range [beg, end).  A range that ends inside a feature group
    // (shared with the next CTA) takes those last n_tail steps FIRST and then runs from its beginning up
    // to that group: both CTAs of a shared group then produce their parts early and the fix-up hides
    // behind the rest of the stream.
    // With clusters: the feature groups [rg_first, g_end) of this cluster, and of each of them the k
    // steps [ks_first, ks_end) of this CTA's rank.
    int beg = 0, end = 0, nsteps = 0, rg_first = 0, ks_first = 0, rg_last = 0, n_tail = 0, g_end = 0, ks_end = 0;
    uint32_t crank = 0;
    if constexpr (CL) {
        crank = cluster_ctarank();
        const int groups = a.total_steps / SPG, nc = (int)cluster_count_x(), cid = (int)cluster_id_x();
        rg_first = (int)(((long long)cid * groups) / nc);
        g_end = (int)(((long long)(cid + 1) * groups) / nc);
        ks_first = (int)crank * SPG / kClusterSize;
        ks_end = ((int)crank + 1) * SPG / kClusterSize;
        nsteps = (g_end - rg_first) * (ks_end - ks_first);
    } else {
        beg = (int)range_begin(cta, ctas, a.total_steps);
        end = (int)range_begin(cta + 1, ctas, a.total_steps);
        nsteps = end - beg;
        rg_first = beg / SPG;
        ks_first = beg - rg_first * SPG;
        rg_last = (end - 1) / SPG;
        n_tail = (end % SPG != 0 && rg_last > rg_first) ? end - rg_last * SPG : 0;
    }
    struct Cursor {
        int rg, ks, i;
    };
    auto cursor_start = [&]() { return n_tail > 0 ? Cursor{rg_last, 0, 0} : Cursor{rg_first, ks_first, 0}; };
    auto cursor_next = [&](Cursor &c) {
        if constexpr (CL) {
            ++c.i;
            if (++c.ks == ks_end) {
                c.ks = ks_first;
                ++c.rg;
            }
        } else {
            if (++c.i == n_tail) {
                c.rg = rg_first;
                c.ks = ks_first;
            } else if (++c.ks == SPG) {
                c.ks = 0;
                ++c.rg;
            }
        }
    };
    // step i (k step ks) is the last one this CTA has of its feature group
    auto part_ends = [&](int i, int ks) { return CL ? ks == ks_end - 1 : (ks == SPG - 1 || i == n_tail - 1 || i == nsteps - 1); };

    if (threadIdx.x == 0) {
        for (int d = 0; d < D; ++d) {
            mbar_init(full_bar(d), 1);
            mbar_init(empty_bar(d), kConsumerWarps);
        }
        mbar_init(cons_bar, kConsumerWarps);
        for (int e = 0; e < 2; ++e) {
            mbar_init(pub_bar(e), kRowBlocks);
            mbar_init(role_bar(e), 1);
        }
        mbar_init(cl_full_bar, kClusterSize);
        mbar_init(cl_done_bar, kClusterSize);
        fence_barrier_init();
        prefetch_tensor_map(&wmap);
        prefetch_tensor_map(&xmap);
    }
    __syncthreads();
    if constexpr (CL) cluster_sync_all();  // no CTA of the cluster is sent an arrival before its barriers exist
    pdl_launch_dependents();

    if (warp == kConsumerWarps) {
        // ======================= producer warp (one lane issues every copy) =======================
        // Weights never depend on the preceding kernel: start them before waiting for it (a routed
        // call must first learn whether it has any row at all).  The stage's barrier gets its one
        // arrival only when the activations are issued, so it cannot complete on weights alone.
        int npre = 0;
        if (lane == 0) {
            if (a.count == nullptr) {
                Cursor c = cursor_start();
                for (; npre < D && npre < nsteps; ++npre) {
                    mbar_expect_tx_only(full_bar(npre), kStepBytes);
                    tma_load_2d(w_stage(npre), &wmap, full_bar(npre), c.ks * 128, c.rg * kTileRows);
                    cursor_next(c);
                }
            }
            pdl_wait();
            const int rows = a.count ? min(*a.count - a.coff, a.M) : a.M;
            if (rows <= 0) return;
            Cursor c = cursor_start();
            for (int i = 0; i < nsteps; ++i) {
                const int d = i % D;
                const int rg = c.rg, ks = c.ks;
                cursor_next(c);
                if (i >= D && !mbar_wait_idle(empty_bar(d), (uint32_t)(((i / D) - 1) & 1), a.status)) break;
                if (i >= npre) {
                    mbar_expect_tx(full_bar(d), kStepBytes + Cfg::X_TX);
                    tma_load_2d(w_stage(d), &wmap, full_bar(d), ks * 128, rg * kTileRows);
                } else {
                    mbar_expect_tx(full_bar(d), Cfg::X_TX);
                }
                // activations of this k range: one [slots x 64] box per 64 k, rows past M read as zero
#pragma unroll
                for (int sb = 0; sb < Geo::X_BOXES; ++sb)
                    tma_load_2d(x_stage(d) + sb * Cfg::X_PITCH, &xmap, full_bar(d), ks * Geo::STEP_K + sb * 64, 0);
            }
        }
        return;
    }

    // CTAs that hold steps of feature group rg_: the first and the last of them
    auto sharers = [&](int rg_, int &c_first, int &c_last) {
        const long long s_first = (long long)rg_ * SPG, s_last = s_first + SPG - 1;
        c_first = (int)(((s_first + 1) * ctas + a.total_steps - 1) / a.total_steps) - 1;
        c_last = (int)(((s_last + 1) * ctas + a.total_steps - 1) / a.total_steps) - 1;
    };

    if (warp == kPublishWarp) {
        // ======================= publishing lane =======================
        // A CTA has at most two parts of shared feature groups: the tail group (taken first) and the
        // group its range starts in.  For each, once k half 0 has stored the part, this lane makes it
        // visible, counts the CTA in and tells the consumers whether they were the last to arrive.  The
        // consumers go on with their next steps meanwhile and only look at the answer at the end.
        if constexpr (CL) return;
        pdl_wait();
        const int rows = a.count ? min(*a.count - a.coff, a.M) : a.M;
        if (rows <= 0 || lane != 0) return;
        const int stop = n_tail > 0 ? rg_last * SPG : end;  // end of the part that starts at `beg`
        const bool head_shared = ks_first > 0 || stop < (rg_first + 1) * SPG;
        const int n_ev = (n_tail > 0 ? 1 : 0) + (head_shared ? 1 : 0);
        const int rg0 = n_tail > 0 ? rg_last : rg_first, rg1 = rg_first;
        // Both counts are issued before either answer is looked at, so that their round trips to
        // the L2 overlap with each other and with the wait for the second part.  The count is one
        // acquire-release atomic (measured faster than fence, atomic, fence).
        int old0 = 0, old1 = 0;
        if (n_ev > 0) {
            if (!mbar_wait(pub_bar(0), 0u, a.status)) return;
            old0 = atom_add_acq_rel(a.counters + (size_t)rg0 * kCounterStride, 1);
        }
        if (n_ev > 1) {
            if (!mbar_wait(pub_bar(1), 0u, a.status)) return;
            old1 = atom_add_acq_rel(a.counters + (size_t)rg1 * kCounterStride, 1);
        }
        for (int e = 0; e < n_ev; ++e) {
            const int rg = e == 0 ? rg0 : rg1;
            int c_first, c_last;
            sharers(rg, c_first, c_last);
            const bool last = (e == 0 ? old0 : old1) == c_last - c_first;
            if (last) a.counters[(size_t)rg * kCounterStride] = 0;  // every sharer has counted in: ready for the next call
            is_last[e] = last ? 1 : 0;
            mbar_arrive(role_bar(e));
        }
        return;
    }

    // ======================= consumer warps =======================
    const int rb = warp % kRowBlocks, kh = warp / kRowBlocks;  // feature block, k half
    const int g = lane >> 2, t = lane & 3;
    const int trow = tile_row_of(g);
    const int K = a.K, N = a.N;
    // Byte offsets of this lane's code chunks inside a weight stage (features rb*16R + r*16 + trow
    // (+8), 128-byte rows, chunk index XOR row % 8) and of its activation chunks inside an
    // activation stage; all fixed for the lifetime of the kernel.
    uint32_t w_off[R][2][GS];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int sg = 0; sg < GS; ++sg) {
                const uint32_t rowb = (uint32_t)((rb * 16 * R + r * 16 + trow + 8 * h) * 128);
                if (BITS == 4 && GS == 2)
                    w_off[r][h][sg] = rowb + ((((uint32_t)(kh * 4 + sg * 2 + (t >> 1))) ^ (uint32_t)trow) << 4) + (uint32_t)((t & 1) * 8);
                else
                    w_off[r][h][sg] = rowb + ((((uint32_t)(kh * 4 + t)) ^ (uint32_t)trow) << 4);
            }
    constexpr int XW = BITS == 4 ? 4 * WPS : (BITS == 8 ? 8 : 4);  // activation words per lane, token and group part
    uint32_t x_off[NT][GS][XW / 4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int sg = 0; sg < GS; ++sg)
#pragma unroll
            for (int i4 = 0; i4 < XW / 4; ++i4) {
                int c;
                if (BITS == 4) c = GS == 1 ? kh * 16 + t * 4 + i4 : kh * 16 + sg * 8 + t * 2 + i4;
                else if (BITS == 8) c = kh * 8 + t * 2 + i4;
                else c = kh * 4 + t;
                x_off[nt][sg][i4] = x_chunk_offset<SLOTS>(c, nt * 8 + g);
            }

    float acc[R][NT][4], accg[R][NT][4];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[r][nt][c] = accg[r][nt][c] = 0.f;

    // Scale and zero point of (feature, group).  Each warp keeps the entries of its own 16R features
    // for the current and the next step in a private shared-memory area: lane l fetches feature l's
    // pair two steps ahead (registers `pend`), packs it as scale << 16 | zero (4-bit: | 0x4300, the
    // bf16 of 128 + zero) one step ahead and every lane then reads the entries of its fragment rows.
    const uint32_t sz_base = base + Cfg::SZ_OFF + (uint32_t)warp * Cfg::SZ_WARP;
    auto sz_fetch = [&](int rg_, int ks_, uint32_t (&dst)[GS][2]) {
        if (!LOWBIT) return;
        const int n = min(rg_ * kTileRows + rb * 16 * R + lane, N - 1);
        const int k0 = ks_ * Geo::STEP_K + kh * Geo::UNIT_K;
#pragma unroll
        for (int sg = 0; sg < GS; ++sg) {
            const int grp = min(group_of_k(k0 + sg * (Geo::UNIT_K / GS)), G - 1);
            dst[sg][0] = __ldg(a.scales + (size_t)n * G + grp);
            dst[sg][1] = __ldg(a.zeros + (size_t)n * G + grp);
        }
    };
    auto sz_store = [&](int slot, const uint32_t (&src)[GS][2]) {
        if (!LOWBIT) return;
#pragma unroll
        for (int sg = 0; sg < GS; ++sg) {
            const uint32_t v = (src[sg][0] << 16) | src[sg][1] | (BITS == 4 ? 0x4300u : 0u);
            if (lane < 16 * R)
                asm volatile("st.shared.u32 [%0], %1;" ::"r"(sz_base + (uint32_t)(((slot * GS + sg) * 16 * R + lane) * 4)), "r"(v) : "memory");
        }
        __syncwarp();
    };
    // The scales and zero points of the first two steps are weights too: fetch them before waiting
    // for the preceding kernel, so that their trip to DRAM is not on the path to the first step.
    uint32_t pend[GS][2], first_sz[GS][2];
    Cursor pf = cursor_start();  // step the next fetch is for
    if (nsteps > 0) {
        sz_fetch(pf.rg, pf.ks, first_sz);
        cursor_next(pf);
    }
    if (nsteps > 1) {
        sz_fetch(pf.rg, pf.ks, pend);
        cursor_next(pf);
    }
    pdl_wait();
    const int rows = a.count ? min(*a.count - a.coff, a.M) : a.M;
    if (rows <= 0) return;
    if (nsteps > 0) sz_store(0, first_sz);

    uint32_t cons_phase = 0;
    int first_ks = -1;  // k step at which this CTA entered the current feature group
    int n_flush = 0, n_shared = 0, shared_rg0 = 0, shared_rg1 = 0;  // flushes so far; parts of shared groups so far
    Cursor cur = cursor_start();
    auto store_y = [&](int n_base, int o, float v) {  // o = slot * 128 + feature within the group
        const int slot = o / kTileRows, n = n_base + o % kTileRows;
        if (slot >= rows || n >= a.N) return;
        const int row = a.idx ? a.idx[slot] : slot;
        if (OUT_F32) reinterpret_cast<float *>(a.Y)[(size_t)row * a.N + n] = v;
        else reinterpret_cast<__nv_bfloat16 *>(a.Y)[(size_t)row * a.N + n] = __float2bfloat16_rn(v);
    };

    auto do_step = [&](int i) -> bool {
        const int d = i % D;
        const int rg = cur.rg, ks = cur.ks;
        cursor_next(cur);
        if (first_ks < 0) first_ks = ks;
        uint32_t fresh_sz[GS][2];
        if (i + 2 < nsteps) {
            sz_fetch(pf.rg, pf.ks, fresh_sz);
            cursor_next(pf);
        }
        // this step's entries for the lane's fragment rows
        uint32_t ent[R][2][GS];
        if (LOWBIT) {
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int sg = 0; sg < GS; ++sg)
                        asm volatile("ld.shared.u32 %0, [%1];"
                                     : "=r"(ent[r][h][sg])
                                     : "r"(sz_base + (uint32_t)((((i & 1) * GS + sg) * 16 * R + r * 16 + trow + 8 * h) * 4)));
        }
        if (!mbar_wait(full_bar(d), (uint32_t)((i / D) & 1), a.status)) return false;
        const int k0 = ks * Geo::STEP_K + kh * Geo::UNIT_K;
        if (k0 < K) {  // warp-uniform: the unit may lie past the end of a ragged row
            const uint32_t ws = w_stage(d), xs = x_stage(d);
#pragma unroll
            for (int sg = 0; sg < GS; ++sg) {
                // ---- this lane's activations, 32-bit words in k order ----
                uint32_t xw[NT][XW];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int i4 = 0; i4 < XW / 4; ++i4) {
                        const uint4 v = lds128(xs + x_off[nt][sg][i4]);
                        xw[nt][4 * i4 + 0] = v.x;
                        xw[nt][4 * i4 + 1] = v.y;
                        xw[nt][4 * i4 + 2] = v.z;
                        xw[nt][4 * i4 + 3] = v.w;
                    }
                // ---- this lane's weights: WPS (4-bit) or 4 words per feature ----
                constexpr int WW = BITS == 4 ? WPS : 4;
                uint32_t wq[R][2][WW];
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (BITS == 4 && GS == 2) {
                            const uint2 v = lds64(ws + w_off[r][h][sg]);
                            wq[r][h][0] = v.x;
                            wq[r][h][WW - 1] = v.y;
                        } else {
                            const uint4 v = lds128(ws + w_off[r][h][sg]);
                            wq[r][h][0] = v.x;
                            wq[r][h][1 % WW] = v.y;
                            wq[r][h][2 % WW] = v.z;
                            wq[r][h][3 % WW] = v.w;
                        }
                    }
                // when every unit ends its quantization group the group sum starts from zero here
                if (CE) {
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                            for (int c = 0; c < 4; ++c) accg[r][nt][c] = 0.f;
                }
                if (BITS == 4) {
                    uint32_t zoff[R][2];
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            zoff[r][h] = prmt(ent[r][h][sg], 0u, 0x1010);  // bf16 of 128 + zero (exact), twice
                        }
#pragma unroll
                    for (int w = 0; w < WW; ++w)
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            // activations in unpack order: (x_p, x_{p+4}) and (x_{p+1}, x_{p+5}), p = 2 hh
                            uint32_t b0[NT], b1[NT];
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt) {
                                const uint32_t r0 = xw[nt][4 * w + hh], r2 = xw[nt][4 * w + 2 + hh];
                                b0[nt] = prmt(r0, r2, 0x5410);
                                b1[nt] = prmt(r0, r2, 0x7632);
                            }
#pragma unroll
                            for (int r = 0; r < R; ++r) {
                                uint32_t av[4];
#pragma unroll
                                for (int h = 0; h < 2; ++h) {
                                    const uint32_t uu = wq[r][h][w];
                                    const uint32_t v0 = lop3_and_or(uu >> (8 * hh), 0x000F000Fu, 0x43004300u);
                                    const uint32_t v1 = lop3_and_or(uu >> (8 * hh + 4), 0x000F000Fu, 0x43004300u);
                                    av[h] = bf16x2_sub(v0, zoff[r][h]);      // codes p, p+4 minus zero
                                    av[2 + h] = bf16x2_sub(v1, zoff[r][h]);  // codes p+1, p+5
                                }
#pragma unroll
                                for (int nt = 0; nt < NT; ++nt)
                                    mma_bf16_16816(accg[r][nt], av[0], av[1], av[2], av[3], b0[nt], b1[nt]);
                            }
                        }
                } else if (BITS == 8) {
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            uint32_t av[4];
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                const float zf = __uint_as_float(0x4B000000u | (ent[r][h][sg] & 0xFFu));  // 2^23 + zero
                                const uint32_t uu = wq[r][h][w];
                                float f[4];
#pragma unroll
                                for (int b = 0; b < 4; ++b)  // (2^23 + byte) - (2^23 + zero) = q - zero exactly
                                    f[b] = __fsub_rn(__uint_as_float(prmt(uu, 0x4B000000u, 0x7650u + (uint32_t)b)), zf);
                                av[h] = pack_bf16x2_rn(f[0], f[1]);  // |q - zero| <= 255: exact in bf16
                                av[2 + h] = pack_bf16x2_rn(f[2], f[3]);
                            }
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt)
                                mma_bf16_16816(accg[r][nt], av[0], av[1], av[2], av[3], xw[nt][2 * w], xw[nt][2 * w + 1]);
                        }
                    }
                } else {
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int p = 0; p < 2; ++p)
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt)
                                mma_bf16_16816(acc[r][nt], wq[r][0][2 * p], wq[r][1][2 * p], wq[r][0][2 * p + 1],
                                               wq[r][1][2 * p + 1], xw[nt][2 * p], xw[nt][2 * p + 1]);
                }
                if (LOWBIT) {
                    // the group sum is complete for this warp when its next unit (one step further)
                    // lies in another group, in another feature group or outside this CTA's range
                    const int kpart = k0 + sg * (Geo::UNIT_K / GS);
                    const bool closes = CE || group_of_k(kpart + Geo::STEP_K) != group_of_k(kpart) || part_ends(i, ks) ||
                                        kpart + Geo::STEP_K >= K;
                    if (closes) {
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            const float s0 = __uint_as_float(ent[r][0][sg] & 0xFFFF0000u);
                            const float s1 = __uint_as_float(ent[r][1][sg] & 0xFFFF0000u);
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt) {
                                acc[r][nt][0] = fmaf(s0, accg[r][nt][0], acc[r][nt][0]);
                                acc[r][nt][1] = fmaf(s0, accg[r][nt][1], acc[r][nt][1]);
                                acc[r][nt][2] = fmaf(s1, accg[r][nt][2], acc[r][nt][2]);
                                acc[r][nt][3] = fmaf(s1, accg[r][nt][3], acc[r][nt][3]);
                                if (!CE) {
#pragma unroll
                                    for (int c = 0; c < 4; ++c) accg[r][nt][c] = 0.f;
                                }
                            }
                        }
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar(d));
        // pack the next step's scale / zero pairs (fetched one step ago) for the whole warp
        if (i + 1 < nsteps) {
            sz_store((i + 1) & 1, pend);
            if (LOWBIT) {
#pragma unroll
                for (int sg = 0; sg < GS; ++sg) {
                    pend[sg][0] = fresh_sz[sg][0];
                    pend[sg][1] = fresh_sz[sg][1];
                }
            }
        }

        // ---- end of this CTA's part of the feature group: combine the k halves and write ----
        if constexpr (CL) {
            if (part_ends(i, ks)) {
                // the sums of both k halves go to this group's place in shared memory, where the
                // cluster picks them up at the end of the round
                float *dst = scratch + (size_t)((rg - rg_first) % a.part_groups) * a.M * kTileRows;
                if (kh == 1) {
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                const int slot = nt * 8 + 2 * t + (c & 1), f = rb * 16 * R + r * 16 + trow + 8 * (c >> 1);
                                if (slot < a.M) dst[slot * kTileRows + f] = acc[r][nt][c];
                            }
                }
                if (!consumer_sync(cons_bar, cons_phase, a.status)) return false;
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const int slot = nt * 8 + 2 * t + (c & 1), f = rb * 16 * R + r * 16 + trow + 8 * (c >> 1);
                            if (kh == 0 && slot < a.M) dst[slot * kTileRows + f] += acc[r][nt][c];
                            acc[r][nt][c] = 0.f;
                        }
            }
            return true;
        }
        if (part_ends(i, ks)) {
            const bool complete = first_ks == 0 && ks == SPG - 1;
            if (!complete && n_shared >= 2) {  // cannot happen: a range has one tail and one head part
                if (a.status) atomicExch(a.status, (int32_t)DMR_ERR_TIMEOUT);  // reported like a wait that ran out
                return false;
            }
            // k half 1 parks its sums (two buffers in turn: the next flush's parking cannot overtake
            // this flush's reading, there is a barrier between them), k half 0 adds them to its own
            float *park = scratch + (n_flush & 1) * Cfg::SUM_FLOATS;
            if (kh == 1) {
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            park[(nt * 8 + 2 * t + (c & 1)) * kTileRows + rb * 16 * R + r * 16 + trow + 8 * (c >> 1)] = acc[r][nt][c];
            }
            if (!consumer_sync(cons_bar, cons_phase, a.status)) return false;
            if (kh == 0) {
                // and writes the outputs (group owned alone) or this CTA's part of a shared group
                const int which = beg > rg * SPG ? 0 : 1;
                float *mine = a.partial + ((size_t)cta * 2 + which) * (kPartSlots * kTileRows);
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const int slot = nt * 8 + 2 * t + (c & 1), f = rb * 16 * R + r * 16 + trow + 8 * (c >> 1);
                            const float v = acc[r][nt][c] + park[slot * kTileRows + f];
                            if (slot >= rows) continue;
                            if (complete) store_y(rg * kTileRows, slot * kTileRows + f, v);
                            else mine[slot * kTileRows + f] = v;
                        }
                if (!complete) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(pub_bar(n_shared));
                }
            }
            if (!complete) {
                if (n_shared == 0) shared_rg0 = rg;
                else shared_rg1 = rg;
                ++n_shared;
            }
            ++n_flush;
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int c = 0; c < 4; ++c) acc[r][nt][c] = 0.f;
            first_ks = -1;
        }
        return true;
    };
    if constexpr (CL) {
        // Rounds of up to part_groups feature groups: every CTA of the cluster streams its k slice of
        // them, then the cluster adds the sums of every output in rank order, each CTA taking its share
        // of the outputs and reading the others' shared memory directly.
        const int my = ks_end - ks_first;
        const uint32_t part_u32 = base + (uint32_t)(D * Cfg::STAGE);
        uint32_t cl_phase = 0;
        int i = 0;
        for (int g0 = rg_first; g0 < g_end; g0 += a.part_groups) {
            const int ng = min(a.part_groups, g_end - g0);
            for (int s = 0; s < ng * my; ++s, ++i)
                if (!do_step(i)) return;
            if (!consumer_sync(cons_bar, cons_phase, a.status)) return;  // this CTA's sums are all in place
            // lane q of the first warp tells CTA q (the arrivals travel side by side)
            if (threadIdx.x < kClusterSize) mbar_arrive_remote(cluster_map(cl_full_bar, threadIdx.x));
            if (!mbar_wait_cluster(cl_full_bar, cl_phase, a.status)) return;
            const int per_group = rows * (kTileRows / 4);  // float4 items of one feature group
            const int items = ng * per_group;
            const int it0 = (int)crank * items / kClusterSize, it1 = ((int)crank + 1) * items / kClusterSize;
            for (int it = it0 + (int)threadIdx.x; it < it1; it += kConsumerWarps * 32) {
                const int gl = it / per_group, rem = it - gl * per_group;
                const int slot = rem >> 5, f4 = rem & 31;
                const uint32_t off = (uint32_t)(((gl * a.M + slot) * kTileRows + f4 * 4) * 4);
                float4 p[kClusterSize];
#pragma unroll
                for (int q = 0; q < kClusterSize; ++q) {
                    const bool has_steps = (q + 1) * SPG / kClusterSize > q * SPG / kClusterSize;
                    p[q] = has_steps ? ld_cluster_f4(cluster_map(part_u32 + off, (uint32_t)q)) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int q = 0; q < kClusterSize; ++q) {
                    v.x += p[q].x;
                    v.y += p[q].y;
                    v.z += p[q].z;
                    v.w += p[q].w;
                }
                const int n_base = (g0 + gl) * kTileRows, o = slot * kTileRows + f4 * 4;
                store_y(n_base, o + 0, v.x);
                store_y(n_base, o + 1, v.y);
                store_y(n_base, o + 2, v.z);
                store_y(n_base, o + 3, v.w);
            }
            // nobody may overwrite its sums (next round) or leave (last round) while others still read them
            if (!consumer_sync(cons_bar, cons_phase, a.status)) return;
            if (threadIdx.x < kClusterSize) mbar_arrive_remote(cluster_map(cl_done_bar, threadIdx.x));
            if (!mbar_wait_cluster(cl_done_bar, cl_phase, a.status)) return;
            cl_phase ^= 1u;
        }
        return;
    }
    for (int i = 0; i < nsteps; ++i)
        if (!do_step(i)) return;

    // ---- shared feature groups this CTA was the last to count into: add all parts in CTA order ----
    const int nvalid4 = rows * (kTileRows / 4);  // float4 items of the rows in use (slot-major)
    for (int e = 0; e < n_shared; ++e) {
        if (!mbar_wait(role_bar(e), 0u, a.status)) return;
        if (is_last[e] == 0) continue;
        const int rg = e == 0 ? shared_rg0 : shared_rg1;
        int c_first, c_last;
        sharers(rg, c_first, c_last);
        const long long s_first = (long long)rg * SPG;
        // loads of up to sixteen parts are in flight together; the additions keep CTA order
        constexpr int PF = NT == 1 ? 12 : 8;
        for (int o4 = threadIdx.x; o4 < nvalid4; o4 += kConsumerWarps * 32) {
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int cj0 = c_first; cj0 <= c_last; cj0 += PF) {
                float4 p[PF];
#pragma unroll
                for (int u = 0; u < PF; ++u) {
                    const int cj = min(cj0 + u, c_last);
                    const int wj = range_begin(cj, ctas, a.total_steps) > s_first ? 0 : 1;
                    p[u] = __ldcg(reinterpret_cast<const float4 *>(a.partial + ((size_t)cj * 2 + wj) * (kPartSlots * kTileRows)) + o4);
                }
#pragma unroll
                for (int u = 0; u < PF; ++u)
                    if (cj0 + u <= c_last) {
                        v.x += p[u].x;
                        v.y += p[u].y;
                        v.z += p[u].z;
                        v.w += p[u].w;
                    }
            }
            store_y(rg * kTileRows, 4 * o4 + 0, v.x);
            store_y(rg * kTileRows, 4 * o4 + 1, v.y);
            store_y(rg * kTileRows, 4 * o4 + 2, v.z);
            store_y(rg * kTileRows, 4 * o4 + 3, v.w);
        }
    }
}

int current_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
    return dev;
}

int sm_count() {
    static int cached[64] = {};
    const int dev = current_device();
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) cached[dev] = n;
        else cached[dev] = 148;
    }
    return cached[dev];
}

// Programmatic dependent launch is on unless the environment says DMR_PDL=0.
bool pdl_enabled() {
    static int v = -1;
    if (v < 0) {
        const char *e = getenv("DMR_PDL");
        v = (e && e[0] == '0') ? 0 : 1;
    }
    return v != 0;
}

// Thread-block clusters are used unless the environment says DMR_CLUSTER=0.
bool cluster_enabled() {
    static int v = -1;
    if (v < 0) {
        const char *e = getenv("DMR_CLUSTER");
        v = (e && e[0] == '0') ? 0 : 1;
    }
    return v != 0;
}

template <int BITS, int NT, int GS, bool CE, bool OUT_F32, bool CL>
dmr_status_t launch_stream_cl(const CUtensorMap &wmap, const CUtensorMap &xmap, StreamArgs a, int ctas, cudaStream_t st,
                              bool *unavailable) {
    using Cfg = StreamCfg<BITS, NT, GS>;
    constexpr int kClusterSize = cluster_size(NT);
    // 227 KB per CTA at most; two resident CTAs must fit into the SM's 228 KB with 1 KB reserved each
    static_assert(Cfg::SMEM <= (NT == 1 ? (228 * 1024 - 2 * 1024) / 2 : 227 * 1024), "stage ring too large");
    static_assert(Cfg::D >= 3, "stage ring too shallow");
    auto kernel = decode_stream_kernel<BITS, NT, GS, CE, OUT_F32, CL>;
    static int configured_on[64] = {};   // 0 = not yet, 1 = ready, -1 = cluster launch not possible on this device
    static int max_clusters_on[64] = {};
    const int dev = current_device();
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(stream_threads(NT, BITS), 1, 1);
    cfg.dynamicSmemBytes = Cfg::SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    if (CL) {
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = kClusterSize;
        attr[n_attr].val.clusterDim.y = 1;
        attr[n_attr].val.clusterDim.z = 1;
        ++n_attr;
    }
    if (configured_on[dev] == 0) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::SMEM);
        if (e != cudaSuccess) {
            g_last_cuda_error = (int)e;
            return DMR_ERR_CUDA;
        }
        configured_on[dev] = 1;
        if (CL) {
            // how many clusters of this kernel the device holds at once (a host-side query, no launch)
            cfg.gridDim = dim3((unsigned)(kClusterSize * 64), 1, 1);
            cfg.attrs = attr;
            cfg.numAttrs = (unsigned)n_attr;
            int n = 0;
            e = cudaOccupancyMaxActiveClusters(&n, kernel, &cfg);
            if (e != cudaSuccess || n < 1) {
                (void)cudaGetLastError();
                configured_on[dev] = -1;
            } else {
                max_clusters_on[dev] = n;
            }
        }
    }
    if (CL) {
        if (configured_on[dev] < 0) {
            *unavailable = true;
            return DMR_OK;
        }
        const int groups = a.total_steps / a.steps_per_group;
        int nc = max_clusters_on[dev];
        if (nc * kClusterSize > kMaxStreamCtas) nc = kMaxStreamCtas / kClusterSize;
        if (nc > groups) nc = groups;
        nc = (groups + (groups + nc - 1) / nc - 1) / ((groups + nc - 1) / nc);  // fewest clusters with the same longest share
        ctas = nc * kClusterSize;
        a.part_groups = (Cfg::PART_BYTES / 4) / (a.M * kTileRows);
        if (a.part_groups < 1) {
            *unavailable = true;
            return DMR_OK;
        }
    }
    cfg.gridDim = dim3((unsigned)ctas, 1, 1);
    if (pdl_enabled()) {
        attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
        ++n_attr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = (unsigned)n_attr;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, wmap, xmap, a);
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        (void)cudaGetLastError();
        return DMR_ERR_CUDA;
    }
    return check_launch();
}

// Cluster mode when the device can hold clusters of this kernel, else the global-memory fix-up.
template <int BITS, int NT, int GS, bool CE, bool OUT_F32>
dmr_status_t launch_stream_t(const CUtensorMap &wmap, const CUtensorMap &xmap, const StreamArgs &a, int ctas,
                             cudaStream_t st) {
    // Clusters pay for small and medium layers, where the sum across CTAs is most of the run time
    // (measured: a 4096 x 4096 INT4 layer takes 6.5 us instead of 10.7).  Large layers keep the contiguous split: a
    // cluster works on whole feature groups, which balances worse, and not every SM can hold its share
    // of a cluster, which the longer streaming phase does not forgive.
    if (cluster_enabled() && a.total_steps <= (BITS == 16 ? kClusterMaxStepsDense : kClusterMaxSteps)) {
        bool unavailable = false;
        const dmr_status_t r = launch_stream_cl<BITS, NT, GS, CE, OUT_F32, true>(wmap, xmap, a, ctas, st, &unavailable);
        if (!unavailable) return r;
    }
    bool unused = false;
    return launch_stream_cl<BITS, NT, GS, CE, OUT_F32, false>(wmap, xmap, a, ctas, st, &unused);
}

template <int BITS, int GS, bool CE>
dmr_status_t launch_stream_nt(const CUtensorMap &wmap, const CUtensorMap &xmap, const StreamArgs &a, int ctas,
                              dmr_out_t out, cudaStream_t st) {
    if (a.tiles == 1) {
        if (out == DMR_OUT_F32) return launch_stream_t<BITS, 1, GS, CE, true>(wmap, xmap, a, ctas, st);
        return launch_stream_t<BITS, 1, GS, CE, false>(wmap, xmap, a, ctas, st);
    }
    if (a.tiles == 4) {
        if (out == DMR_OUT_F32) return launch_stream_t<BITS, 4, GS, CE, true>(wmap, xmap, a, ctas, st);
        return launch_stream_t<BITS, 4, GS, CE, false>(wmap, xmap, a, ctas, st);
    }
    if (out == DMR_OUT_F32) return launch_stream_t<BITS, 2, GS, CE, true>(wmap, xmap, a, ctas, st);
    return launch_stream_t<BITS, 2, GS, CE, false>(wmap, xmap, a, ctas, st);
}

}  // namespace

size_t stream_scratch_bytes(int N) {
    const size_t groups = (size_t)(N + kTileRows - 1) / kTileRows;
    return kStreamPartialBytes + groups * kCounterStride * sizeof(int32_t);
}

void stream_plan(int M, int N, int K, int bits, int *tiles, long long *steps, int *cluster) {
    const int step_k = 1024 / bits;
    *tiles = M <= 8 ? 1 : (M <= 16 ? 2 : 4);
    *steps = (long long)((N + kTileRows - 1) / kTileRows) * ((K + step_k - 1) / step_k);
    *cluster = (cluster_enabled() && *steps <= (bits == 16 ? kClusterMaxStepsDense : kClusterMaxSteps)) ? cluster_size(*tiles) : 0;
}

bool stream_supported(int M, int N, int K, int bits /*16 = bf16 weights*/, int g) {
    (void)N;
    if (M < 1 || M > 32) return false;
    if (bits == 16) return K % 8 == 0;
    if (bits == 4) return g % 128 == 0 || g == 64;
    if (bits == 8) return g % 64 == 0;
    return false;
}

dmr_status_t launch_stream(const uint16_t *X, int M, RowSel sel, const void *weights, const uint16_t *scales,
                           const uint8_t *zeros, int N, int K, int bits, int g, void *Y, dmr_out_t out,
                           void *scratch, int32_t *status, cudaStream_t st, int batch_rows) {
    const int step_k = 1024 / bits;
    StreamArgs a;
    const int call_rows = batch_rows > M ? batch_rows : M;
    a.tiles = call_rows <= 8 ? 1 : (call_rows <= 16 ? 2 : 4);
    a.idx = sel.idx;
    a.count = sel.count;
    a.scales = scales;
    a.zeros = zeros;
    a.Y = Y;
    const size_t groups = (size_t)(N + kTileRows - 1) / kTileRows;
    // The partial sums come first (a fixed size) and the counters after them, so that a counter's address never
    // depends on N: layers of different widths can share one scratch area without one layer's partial sums
    // landing on words that another layer needs to find zero.
    a.partial = reinterpret_cast<float *>(scratch);
    a.counters = reinterpret_cast<int32_t *>(reinterpret_cast<char *>(scratch) + kStreamPartialBytes);
    a.status = status;
    a.M = M;
    a.coff = sel.offset;
    a.N = N;
    a.K = K;
    a.g_size = bits == 16 ? K : g;
    a.g_shift = -1;
    for (int sh = 0; sh < 31; ++sh)
        if ((1 << sh) == a.g_size) a.g_shift = sh;
    a.steps_per_group = (K + step_k - 1) / step_k;
    const long long total = (long long)groups * a.steps_per_group;
    if (total > 0x7FFFFFFF) return DMR_ERR_UNSUPPORTED;
    a.total_steps = (int)total;
    a.part_groups = 0;
    int ctas = sm_count() * (a.tiles == 1 ? 2 : 1);  // the 8-row kernels fit twice on an SM
    if (a.tiles == 4 && ctas > kMaxStreamCtas / 2) ctas = kMaxStreamCtas / 2;  // 32-slot parts are twice as large
    if (ctas > kMaxStreamCtas) ctas = kMaxStreamCtas;
    if (ctas > a.total_steps) ctas = a.total_steps;
    CUtensorMap wmap;
    const uint64_t row_bytes = (uint64_t)K * bits / 8;
    if (!make_tensor_map_2d(&wmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, weights, (uint64_t)N, row_bytes, row_bytes, kTileRows,
                            128, TmaSwizzle::k128B))
        return DMR_ERR_CUDA;
    // X holds M consecutive rows (for a routed call: the gathered rows); box = [8 or 16 slots][64 k]
    CUtensorMap xmap;
    if (!make_tensor_map_2d(&xmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, (uint64_t)M, (uint64_t)K, (uint64_t)K * 2,
                            8 * a.tiles, 64, TmaSwizzle::k128B))
        return DMR_ERR_CUDA;
    if (bits == 16) return launch_stream_nt<16, 1, false>(wmap, xmap, a, ctas, out, st);
    if (bits == 8) {
        if (g == 64) return launch_stream_nt<8, 1, true>(wmap, xmap, a, ctas, out, st);
        return launch_stream_nt<8, 1, false>(wmap, xmap, a, ctas, out, st);
    }
    if (g == 64) return launch_stream_nt<4, 2, true>(wmap, xmap, a, ctas, out, st);
    if (g == 128) return launch_stream_nt<4, 1, true>(wmap, xmap, a, ctas, out, st);
    return launch_stream_nt<4, 1, false>(wmap, xmap, a, ctas, out, st);
}

}  // namespace dmr
