// Projection with the multiply-adds on the 5th-generation tensor cores (tcgen05 + tensor memory).
//
// For many machines the projection P = G Xi^T is a dense contraction whose operand Xi is generated on
// the fly.  A CTA (8 warps) owns 128 or 256 vectors (one or two groups of 128, the M of the instruction)
// and a range of coordinates.  Per stage (its vectors x 32 coordinates) every thread generates four or
// eight counters' worth of Gaussians (one coordinate block, 4 or 8 vectors), splits each value into a tf32
// head and tail (z = hi + lo, both exact in fp32) and writes the two planes to shared memory in the
// K-major core-matrix layout the tensor core reads; in turn the warps also stage the machines' gradients
// for the same 32 coordinates (split the same way when they are fp32; bf16 is exact in tf32).  The
// products of stage c are issued by one elected lane of warp c % 8 once it has finished generating stage
// c + 1 (and before it reports that stage done, which keeps the issue order equal to the stage order); the
// descriptors are computed by the whole warp from warp-uniform values, so they stay in uniform registers.
// Per group of 128 vectors and 8 coordinates:  tcgen05.mma  D[128 vectors x N machines] += A[128 x 8] *
// B[8 x N]  (N = 16, 32 or 64) for hi*hi, lo*hi (and hi*lo for fp32 gradients).  D lives in tensor
// memory, double buffered, with the small products in an accumulator of their own: every 8 stages (256
// coordinates) the warps move both to registers with tcgen05.ld (a piece of 32 vectors x 16 machines at a
// time) and add them to fp32 running sums.  The tensor core's accumulator loses about half an ulp
// of the running sum per product, always in the same direction, so its chains are kept short and the
// large and small terms apart.  Stage buffers and accumulators are handed over with mbarriers; every
// wait is bounded, and a wait that runs out sets a device status word and lets the CTA leave through the
// normal exit (which releases its tensor memory).  The per-CTA partial sums have the layout of the
// scalar kernel.
#include "core_internal.h"

#include <cuda_bf16.h>

#include <utility>

namespace core {

namespace {

constexpr int kTcWarps = 8;
constexpr int kTcThreads = 32 * kTcWarps;
constexpr int kTcVectors = 128;                 // M of the instruction = vectors per group (a CTA owns VG groups)
constexpr int kTcMaxN = 64;                     // largest N of the instruction = machines per pass (16, 32 or 64)
constexpr int kTcMinMachines = 9;               // fewer machines: the scalar kernel is used
constexpr int kTcStageBlocks = 8;               // coordinate blocks per stage: 32 coordinates = 128 B per row
constexpr int kTcTileStages = 8;                // stages between two drains of the accumulators
constexpr int kTcTileBlocks = kTcStageBlocks * kTcTileStages;       // 64 blocks = 256 coordinates
// Geometry that depends on N (machines per pass: 16, 32 or 64; 64 with two groups only), on the gradients' type and on VG (groups of
// 128 vectors per CTA).  bf16 gradients are exact in tf32 and need one plane, fp32 gradients a head and a
// tail plane.  With one group two CTAs share an SM (about 113 KB of shared memory each); with two groups a
// CTA has the SM to itself, every thread generates eight counters per stage instead of four, and the
// per-stage work that does not depend on the number of vectors (hand-over, issue, staging of the
// gradients) is spread over twice as many Gaussians.
template <int NT, bool BF16, int VG>
struct TcShape {
    static constexpr uint32_t kPlaneA = VG * kTcVectors * 128;         // bytes of one plane of Xi per stage
    static constexpr uint32_t kPlaneB = NT * 128;                      // bytes of one plane of G per stage
    static constexpr int kPlanesB = BF16 ? 1 : 2;
    static constexpr uint32_t kStageBytes = 2 * kPlaneA + kPlanesB * kPlaneB;
    static constexpr uint32_t kBudget = (VG == 1 ? 113u : 226u) * 1024u;
    static constexpr int kStages = 3 * kStageBytes + 2048 <= kBudget ? 3 : 2;
    static constexpr uint32_t kSmemBytes = kStages * kStageBytes + 128 + 1024;   // + barriers + alignment slack
    static constexpr uint32_t kTmemColumns = 4 * NT * VG;              // two buffers x groups x (head, tail products) x N
    // A draining warp reads its quarter of the tensor-memory lanes (32 vectors of a group) x 16 columns
    // (machines): VG * NT / 16 such pieces per quarter, shared out over one or two warps per quarter.
    static constexpr int kPieces = VG * NT / 16;
    static constexpr int kDrainWarps = kPieces > 1 ? 8 : 4;
    static constexpr int kPiecesPerWarp = kPieces > 2 ? kPieces / 2 : 1;
    // Staging of the gradients: 16-byte pieces per stage, one or two per thread of the warps on duty.
    static constexpr int kPiecesB = NT * (BF16 ? 4 : 8);
    static constexpr int kDutyWarps = kPiecesB / 32 < kTcWarps ? kPiecesB / 32 : kTcWarps;
    static constexpr int kDutyPieces = kPiecesB / (32 * kDutyWarps);   // per thread on duty
    // Instruction descriptor: fp32 accumulator (1 at bit 4), tf32 A and B (2 at bits 7 and 10), both
    // K-major, N >> 3 at bit 17, M >> 4 at bit 24.
    static constexpr uint32_t kIdesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(NT >> 3) << 17) |
                                       ((uint32_t)(kTcVectors >> 4) << 24);
};
constexpr uint64_t kTcWaitLimitNs = 100ull * 1000 * 1000;   // a wait gives up after 100 ms of the global timer

__device__ int g_tc_status;                     // 0, or the code of a wait that ran out

struct TcArgs {
    const void *G;
    int64_t ldg;
    int64_t d;
    int64_t tiles;
    uint64_t q_base;
    float *partial;
    int n;
    int m;
    int aligned;
    uint32_t t;
    RoundKeys keys;
};

// ---- thin wrappers over the PTX this kernel needs --------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: false when the phase did not complete within limit_ns of the global timer (read only
// once a first probe has failed, so a wait that is served at once costs one probe).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint64_t limit_ns = kTcWaitLimitNs) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    do {
#pragma unroll 1
        for (int probe = 0; probe < 64; ++probe)
            if (mbar_try_wait(bar, parity)) return true;
    } while (global_timer_ns() - t0 < limit_ns);
    return false;
}
// True in exactly one lane of a converged warp.  Unlike a test of the lane index this keeps the branch, and the
// operands computed for the instructions under it, warp-uniform in the compiler's eyes.
__device__ __forceinline__ bool elect_one() {
    uint32_t chosen;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(chosen));
    return chosen != 0;
}
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t slot, uint32_t columns) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(columns) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_free(uint32_t taddr, uint32_t columns) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(columns) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], tf32 operands, fp32 accumulate, M = 128, N = 16, K = 8.
// The descriptors arrive as (low word, high word): only the low word (address field) varies.
__device__ __forceinline__ void tc_mma_tf32(uint32_t d_tmem, uint32_t a_lo32, uint32_t b_lo32, uint32_t desc_hi32,
                                            uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], da, db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo32), "r"(b_lo32), "r"(desc_hi32), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 16 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_load16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int c = 0; c < 16; ++c) v[c] = __uint_as_float(r[c]);
}
template <uint32_t OFFSET = 0>
__device__ __forceinline__ void st_shared_v4(uint32_t addr, float x, float y, float z, float w) {
    asm volatile("st.shared.v4.f32 [%0+%5], {%1, %2, %3, %4};" ::"r"(addr), "f"(x), "f"(y), "f"(z), "f"(w), "n"(OFFSET)
                 : "memory");
}

// Shared-memory matrix descriptor, K-major, no swizzle: a core matrix is 8 rows x 16 bytes stored
// contiguously (128 B); the two core matrices of one instruction along K are `kLbo` bytes apart, groups
// of eight rows `kSbo` bytes apart.  Fields: address >> 4 at bit 0, kLbo >> 4 at bit 16, kSbo >> 4 at
// bit 32, descriptor version 1 at bit 46, layout type 0 (no swizzle) at bit 61.
constexpr uint32_t kLbo = 128;
constexpr uint32_t kSbo = 128 * kTcStageBlocks;    // 1024: eight 16-byte chunks per row
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t addr) { return ((addr & 0x3FFFFu) >> 4) | ((kLbo >> 4) << 16); }
constexpr uint32_t kDescHi = (kSbo >> 4) | (1u << 14);
// Byte offset of the 16-byte chunk (row, c) inside a plane.
__device__ __forceinline__ uint32_t plane_offset(int row, int c) {
    return (uint32_t)(row >> 3) * kSbo + (uint32_t)c * kLbo + (uint32_t)(row & 7) * 16u;
}

__device__ __forceinline__ float tf32_head(float x) { return __uint_as_float(__float_as_uint(x) & 0xFFFFE000u); }

// Head and tail of the four Gaussians of vector (lane + 32 U) into the two planes (PLANE_A bytes apart)
// of a stage.
template <int U, uint32_t PLANE_A>
__device__ __forceinline__ void store_split(uint32_t dst, const float4 &z) {
    const float hx = tf32_head(z.x), hy = tf32_head(z.y), hz = tf32_head(z.z), hw = tf32_head(z.w);
    st_shared_v4<U * 4 * kSbo>(dst, hx, hy, hz, hw);
    st_shared_v4<U * 4 * kSbo + PLANE_A>(dst, z.x - hx, z.y - hy, z.z - hz, z.w - hw);
}
template <uint32_t PLANE_A, int... U>
__device__ __forceinline__ void store_split_all(uint32_t dst, const float4 *z, std::integer_sequence<int, U...>) {
    (store_split<U, PLANE_A>(dst, z[U]), ...);
}

// Head and tail of four fp32 gradient values into the two G planes (PLANE_B bytes apart) of a stage.
template <uint32_t PLANE_B>
__device__ __forceinline__ void store_split_b(uint32_t dst, float x, float y, float z, float w) {
    const float hx = tf32_head(x), hy = tf32_head(y), hz = tf32_head(z), hw = tf32_head(w);
    st_shared_v4(dst, hx, hy, hz, hw);
    st_shared_v4<PLANE_B>(dst, x - hx, y - hy, z - hz, w - hw);
}

// One thread's piece of a ragged or unaligned stage (4 coordinates for fp32, 8 for bf16, from k0 on),
// element by element, zero beyond d and beyond n.  Kept out of line: it is rare.
template <typename GT, uint32_t PLANE_B>
__device__ __noinline__ void stage_piece_slowly(const GT *G, int64_t ldg, int64_t d, int n, int i, int64_t k0, uint32_t dst) {
    constexpr bool BF16 = sizeof(GT) == 2;
    for (int part = 0; part < (BF16 ? 2 : 1); ++part) {
        float vals[4] = {0.f, 0.f, 0.f, 0.f};
        if (i < n) {
#pragma unroll
            for (int l = 0; l < 4; ++l) {
                const int64_t k = k0 + 4 * part + l;
                if (k < d) {
                    if constexpr (BF16)
                        vals[l] = __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short *>(G) + (int64_t)i * ldg + k) << 16);
                    else
                        vals[l] = __ldg(reinterpret_cast<const float *>(G) + (int64_t)i * ldg + k);
                }
            }
        }
        if constexpr (BF16)
            st_shared_v4(dst + (uint32_t)part * kLbo, vals[0], vals[1], vals[2], vals[3]);
        else
            store_split_b<PLANE_B>(dst, vals[0], vals[1], vals[2], vals[3]);
    }
}

template <typename GT, int NT, int VG>
__global__ void __launch_bounds__(kTcThreads, VG == 1 ? 2 : 1)
project_tc_kernel(const __grid_constant__ TcArgs a) {
    constexpr bool BF16 = sizeof(GT) == 2;
    using Shape = TcShape<NT, BF16, VG>;
    constexpr int kTcStages = Shape::kStages;
    constexpr uint32_t kTcStageBytes = Shape::kStageBytes, kTcPlaneA = Shape::kPlaneA, kTcPlaneB = Shape::kPlaneB;
    constexpr uint32_t kTcTmemColumns = Shape::kTmemColumns, kIdesc = Shape::kIdesc;
    constexpr int kDrainWarps = Shape::kDrainWarps, kPiecesPerWarp = Shape::kPiecesPerWarp;
    constexpr int kCalls = 4 * VG;                                   // counters per thread and stage
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;                    // stage buffers, 1024-byte aligned
    unsigned char *const smem = smem_raw + (base - raw);
    const uint32_t bars = base + kTcStages * kTcStageBytes;
    const uint32_t bar_full = bars, bar_empty = bars + 8 * kTcStages;
    const uint32_t bar_acc_full = bars + 16 * kTcStages, bar_acc_empty = bar_acc_full + 16, bar_done = bar_acc_full + 32;
    volatile uint32_t *const words = reinterpret_cast<volatile uint32_t *>(smem + kTcStages * kTcStageBytes + 16 * kTcStages + 40);
    volatile uint32_t *const tmem_slot = words;                      // written by tcgen05.alloc
    volatile uint32_t *const abort_flag = words + 1;

    const int tid = threadIdx.x, lane = tid & 31;
    // the warp's index, broadcast from a lane so that the compiler knows it to be the same in all lanes
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const GT *G = static_cast<const GT *>(a.G);

    if (tid == 0) {
        for (int s = 0; s < kTcStages; ++s) {
            mbar_init(bar_full + 8 * s, kTcThreads);                 // one arrival per thread
            mbar_init(bar_empty + 8 * s, 1);                         // tcgen05.commit of the stage's products
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_acc_full + 8 * b, kTcTileStages);          // one tcgen05.commit per stage of the tile
            mbar_init(bar_acc_empty + 8 * b, kDrainWarps);           // one arrival per draining warp
        }
        mbar_init(bar_done, kTcWarps);                               // one tcgen05.commit per warp at the end
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 0) tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), kTcTmemColumns);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t taddr = __shfl_sync(0xffffffffu, *tmem_slot, 0);

    const int64_t per = (a.tiles + gridDim.x - 1) / gridDim.x;
    const int64_t tile_begin = (int64_t)blockIdx.x * per;
    const int64_t tile_end = min(tile_begin + per, a.tiles);
    auto stages_of = [&](int64_t tile) {
        const int64_t left = a.d - tile * (4 * kTcTileBlocks);
        const int64_t st = (left + 4 * kTcStageBlocks - 1) / (4 * kTcStageBlocks);
        return (int)(st < kTcTileStages ? st : kTcTileStages);
    };
    auto give_up = [&](int code) {
        *abort_flag = 1;
        atomicMax(&g_tc_status, code);
    };
    // Whole-warp wait.  The common case (the phase completed long ago) costs one probe and one vote.
    // Has any warp of this CTA given up?  One answer for the whole warp: a flag raised between two lanes'
    // reads must not split the warp (the lanes that stayed would wait for the ones that left).
    auto aborted = [&]() { return __any_sync(0xffffffffu, *abort_flag != 0); };
    // Whole-warp wait.  The common case (the phase completed long ago) costs one probe and one vote.
    auto warp_wait = [&](uint32_t bar, uint32_t parity, int code) {
        if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
        bool ok = !aborted();
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar, parity));
        if (!ok && lane == 0) give_up(code);
        return ok;
    };
    // A draining warp owns pieces of 32 vectors (its quarter of the tensor-memory lanes, in one group) x
    // 16 machines: piece index = group * (NT / 16) + half of the columns.  With one piece per quarter
    // warps 0..3 drain; with two, warps 4..7 take the second; with four, each warp takes two.
    float outer[kPiecesPerWarp][16];
#pragma unroll
    for (int r = 0; r < kPiecesPerWarp; ++r)
#pragma unroll
        for (int c = 0; c < 16; ++c) outer[r][c] = 0.f;
    const int piece0 = (warp >> 2) * kPiecesPerWarp;                 // first piece of this warp
    const int jbase = blockIdx.y * (VG * kTcVectors) + lane;         // this thread's vectors: jbase + 32 u
    auto drain = [&](int64_t local_tile) {                           // draining warps: tensor memory -> running sums
        const uint32_t b = (uint32_t)(local_tile & 1);
        if (!warp_wait(bar_acc_full + 8 * b, (uint32_t)((local_tile >> 1) & 1), 3)) return;
        tc_fence_after_sync();
#pragma unroll
        for (int r = 0; r < kPiecesPerWarp; ++r) {
            const int piece = piece0 + r, g = piece / (NT / 16), half = piece % (NT / 16);
            float head[16], tail[16];
            const uint32_t lane_base = taddr + ((uint32_t)((warp & 3) * 32) << 16) + (b * VG + (uint32_t)g) * (2 * NT) +
                                       (uint32_t)half * 16u;
            tmem_load16(lane_base, head);
            tmem_load16(lane_base + NT, tail);
#pragma unroll
            for (int c = 0; c < 16; ++c) outer[r][c] += head[c] + tail[c];
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_acc_empty + 8 * b);
    };

    // Gradient staging is shared out among the warps in turn: DUTY warps serve a stage, one 16-byte piece
    // per thread, fetched one stage ahead so that the load is in flight while the previous stage is
    // generated.
    constexpr int DUTY = Shape::kDutyWarps;                          // warps on duty per stage
    constexpr int PPT = Shape::kDutyPieces;                           // 16-byte pieces per thread on duty (1 or 2)
    constexpr uint32_t ROTA = kTcWarps / DUTY;                        // stages until a warp's turn comes again
    const uint32_t duty_phase = (uint32_t)warp / DUTY;                // serves stages c with c % ROTA == duty_phase
    const uint32_t fetch_phase = (duty_phase + ROTA - 1) % ROTA;      // and fetches for them one stage earlier
    const int64_t range_begin = tile_begin * (int64_t)(4 * kTcTileBlocks);
    const int64_t range_end = min(tile_end * (int64_t)(4 * kTcTileBlocks), a.d);
    // stages of this CTA: the first `fast_stages` lie wholly inside d and can be read 16 bytes at a time
    const uint32_t total_stages = range_end > range_begin ? (uint32_t)((range_end - range_begin + 31) >> 5) : 0u;
    const uint32_t fast_stages = a.aligned && range_end > range_begin ? (uint32_t)((range_end - range_begin) >> 5) : 0u;
    int duty_i[PPT], duty_c[PPT];                                     // machine, piece of the machine's row
    uint32_t duty_off[PPT];
    const GT *duty_src[PPT];
    uint4 held[PPT];
#pragma unroll
    for (int r = 0; r < PPT; ++r) {
        const int piece = ((warp % DUTY) * 32 + lane) + r * (DUTY * 32);   // always the same pieces of the stage
        duty_i[r] = BF16 ? piece >> 2 : piece >> 3;
        duty_c[r] = BF16 ? piece & 3 : piece & 7;
        duty_off[r] = 2 * kTcPlaneA + plane_offset(duty_i[r], BF16 ? 2 * duty_c[r] : duty_c[r]);
        duty_src[r] = G + (int64_t)duty_i[r] * a.ldg + range_begin + (BF16 ? 8 : 4) * duty_c[r];
        held[r] = make_uint4(0, 0, 0, 0);
    }
    auto fetch = [&](uint32_t c) {                                    // pieces of stage c, if they can be read whole
        if (c < fast_stages) {
#pragma unroll
            for (int r = 0; r < PPT; ++r)
                if (duty_i[r] < a.n) held[r] = __ldg(reinterpret_cast<const uint4 *>(duty_src[r] + (int64_t)c * 32));
        }
    };
    auto deposit = [&](uint32_t c, uint32_t sb) {                     // stage c into the buffer at sb
#pragma unroll
        for (int r = 0; r < PPT; ++r) {
            const uint32_t dst = sb + duty_off[r];
            if (c < fast_stages) {
                const uint4 h = duty_i[r] < a.n ? held[r] : make_uint4(0, 0, 0, 0);
                if constexpr (BF16) {
                    st_shared_v4(dst, __uint_as_float(h.x << 16), __uint_as_float(h.x & 0xFFFF0000u),
                                 __uint_as_float(h.y << 16), __uint_as_float(h.y & 0xFFFF0000u));
                    st_shared_v4<kLbo>(dst, __uint_as_float(h.z << 16), __uint_as_float(h.z & 0xFFFF0000u),
                                       __uint_as_float(h.w << 16), __uint_as_float(h.w & 0xFFFF0000u));
                } else {
                    store_split_b<kTcPlaneB>(dst, __uint_as_float(h.x), __uint_as_float(h.y), __uint_as_float(h.z), __uint_as_float(h.w));
                }
            } else {
                stage_piece_slowly<GT, kTcPlaneB>(G, a.ldg, a.d, a.n, duty_i[r],
                                                  range_begin + (int64_t)c * 32 + (BF16 ? 8 : 4) * duty_c[r], dst);
            }
        }
    };

    // Products of one finished stage, issued by one lane.  `st` is the stage's index in its tile of
    // `stages`, `local` the tile's index in this CTA, (slot, parity) its ring position.
    auto issue = [&](uint32_t slot, uint32_t parity, int st, int stages, int64_t local) {
        const uint32_t b = (uint32_t)(local & 1);
        bool ok = true;
        // the accumulators are free once the tile two back has been drained
        if (st == 0) ok = warp_wait(bar_acc_empty + 8 * b, (uint32_t)(((local >> 1) & 1) ^ 1), 4);
        if (ok) ok = warp_wait(bar_full + 8 * slot, parity, 5);
        if (ok) {
            tc_fence_after_sync();
            // Everything up to the instructions themselves is computed by the whole warp from values that are
            // the same in all lanes (descriptors then stay in uniform registers); one elected lane issues.
            // Products with the head of xi and the head of g go to one accumulator, the small products (a
            // tail times a head) to another: the tensor core's accumulation error scales with the running
            // sum, and the small ones then cost nothing.
            const uint32_t a_hi0 = smem_desc_lo(base + slot * kTcStageBytes);             // other planes: + bytes >> 4
            const uint32_t b_hi = a_hi0 + (2 * kTcPlaneA >> 4), b_lo = b_hi + (kTcPlaneB >> 4);
            if (elect_one()) {
#pragma unroll
                for (int g = 0; g < VG; ++g) {
                    const uint32_t d_head = taddr + (b * VG + (uint32_t)g) * (2 * NT), d_tail = d_head + NT;
                    const uint32_t a_hi = a_hi0 + (uint32_t)g * (kTcVectors * 128u >> 4), a_lo = a_hi + (kTcPlaneA >> 4);
#pragma unroll
                    for (int kk = 0; kk < kTcStageBlocks / 2; ++kk) {
                        const uint32_t step = (uint32_t)kk * 2u * kLbo >> 4;
                        const uint32_t more = (st | kk) != 0;
                        tc_mma_tf32(d_head, a_hi + step, b_hi + step, kDescHi, kIdesc, more);
                        tc_mma_tf32(d_tail, a_lo + step, b_hi + step, kDescHi, kIdesc, more);
                        if constexpr (!BF16) tc_mma_tf32(d_tail, a_hi + step, b_lo + step, kDescHi, kIdesc, 1u);
                    }
                }
                tc_commit(bar_empty + 8 * slot);                      // the stage buffer may be refilled
                tc_commit(bar_acc_full + 8 * b);                      // one of the tile's kTcTileStages arrivals
                if (st + 1 == stages)                                 // a short last tile: make up the count
                    for (int r = stages; r < kTcTileStages; ++r) tc_commit(bar_acc_full + 8 * b);
            }
            tc_fence_before_sync();                                   // issued before this warp's arrival below
        }
        __syncwarp();
    };

    const uint32_t row_off = plane_offset(lane, warp);               // chunk of vector `lane`; vector lane + 32 u is 4 u row groups on
    uint32_t s = 0, ph = 0;                                          // ring position and its parity
    uint32_t count = 0;                                              // stages done
    // the stage before the current one, whose products are issued by warp (count - 1) % 8
    uint32_t prev_s = 0, prev_ph = 0;
    int prev_st = 0, prev_stages = 0;
    int64_t prev_local = 0;
    uint32_t q_hi = (uint32_t)((a.q_base + (uint64_t)tile_begin * kTcTileBlocks) >> 32);
    JPart jp[kCalls];
#pragma unroll
    for (int u = 0; u < kCalls; ++u) jp[u] = philox_jpart((uint32_t)(jbase + 32 * u), q_hi, a.keys);
    if (duty_phase == 0) fetch(0);
    bool alive = true;
    for (int64_t tile = tile_begin; tile < tile_end && alive; ++tile) {
        const uint64_t q_tile = a.q_base + (uint64_t)tile * kTcTileBlocks;
        if ((uint32_t)(q_tile >> 32) != q_hi) {                      // once per 2^32 blocks
            q_hi = (uint32_t)(q_tile >> 32);
#pragma unroll
            for (int u = 0; u < kCalls; ++u) jp[u] = philox_jpart((uint32_t)(jbase + 32 * u), q_hi, a.keys);
        }
        const int stages = stages_of(tile);
        uint32_t q_lo = (uint32_t)q_tile + (uint32_t)warp;
        for (int st = 0; st < stages; ++st, q_lo += kTcStageBlocks, ++count) {
            if (!warp_wait(bar_empty + 8 * s, ph ^ 1u, 1)) { alive = false; break; }
            const uint32_t sb = base + s * kTcStageBytes;
            {
                const uint32_t turn = count % ROTA;
                if (turn == duty_phase) deposit(count, sb);
                if (turn == fetch_phase && count + 1 < total_stages) fetch(count + 1);   // the same turn when all warps are on duty
            }
            const QPart qp = philox_qpart(q_lo, a.t, a.keys);
            uint4 w[kCalls];
#pragma unroll
            for (int u = 0; u < kCalls; ++u) w[u] = philox_combine(jp[u], qp, a.keys);
            float4 z[kCalls];
            box_muller4xN<kCalls>(w, z);
            store_split_all<kTcPlaneA>(sb + row_off, z, std::make_integer_sequence<int, kCalls>{});
            // The previous stage's products go out before this warp reports the current stage done, so
            // that no other warp can be issuing a later stage first.
            if (count > 0 && (uint32_t)warp == ((count - 1) & (kTcWarps - 1))) {
                issue(prev_s, prev_ph, prev_st, prev_stages, prev_local);
                if (aborted()) { alive = false; break; }
            }
            fence_proxy_async_smem();                                // my stores, visible to the tensor core
            mbar_arrive(bar_full + 8 * s);
            prev_s = s; prev_ph = ph; prev_st = st; prev_stages = stages; prev_local = tile - tile_begin;
            if (++s == kTcStages) { s = 0; ph ^= 1u; }
        }
        // the tile before this one has long been multiplied: fold it in while this one is in flight
        if (alive && warp < kDrainWarps && tile > tile_begin) drain(tile - tile_begin - 1);
    }
    if (alive && count > 0 && (uint32_t)warp == ((count - 1) & (kTcWarps - 1)))
        issue(prev_s, prev_ph, prev_st, prev_stages, prev_local);
    if (alive && warp < kDrainWarps && tile_end > tile_begin) drain(tile_end - tile_begin - 1);

    if (warp < kDrainWarps) {
#pragma unroll
        for (int r = 0; r < kPiecesPerWarp; ++r) {
            const int piece = piece0 + r, g = piece / (NT / 16), half = piece % (NT / 16);
            const int j = blockIdx.y * (VG * kTcVectors) + g * kTcVectors + (warp & 3) * 32 + lane;
            if (j < a.m) {
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const int i = half * 16 + c;
                    if (i < a.n) a.partial[((int64_t)blockIdx.x * a.n + i) * a.m + j] = outer[r][c];
                }
            }
        }
    }

    // nothing of this CTA may still be running on the tensor core when its tensor memory goes back
    if (elect_one()) tc_commit(bar_done);                            // the lane that issued this warp's products
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        if (lane == 0 && !mbar_wait(bar_done, 0)) give_up(6);
        __syncwarp();
        tc_fence_after_sync();
        tmem_free(taddr, kTcTmemColumns);
    }
}

// Test kernel for the bounded waits: two warps share a barrier that expects one arrival nobody makes.
// Warp 0 waits on it with the helper the projection uses (and a short limit), records the code when the
// wait runs out and raises the CTA's abort flag; warp 1 watches the flag the way the projection's warps
// do.  Both leave by the normal exit.  No tensor-core instruction, no tensor memory.
__global__ void wait_timeout_probe_kernel(uint64_t limit_ns, int code, uint32_t *observed) {
    __shared__ __align__(8) unsigned long long barrier_word;
    __shared__ volatile uint32_t abort_flag;
    const uint32_t bar = smem_u32(&barrier_word);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (warp == 0) {
        const bool ok = __all_sync(0xffffffffu, mbar_wait(bar, 0, limit_ns));
        if (!ok && lane == 0) {
            abort_flag = 1;
            atomicMax(&g_tc_status, code);
        }
        if (lane == 0) observed[0] = ok ? 1u : 0u;
    } else {
        // bounded too: at most ten times the limit
        const uint64_t t0 = global_timer_ns();
        bool seen = false;
        for (;;) {                                                   // both votes are taken by the whole warp
            seen = __any_sync(0xffffffffu, abort_flag != 0);
            const bool time_up = __any_sync(0xffffffffu, global_timer_ns() - t0 >= 10 * limit_ns);
            if (seen || time_up) break;
        }
        if (lane == 0) observed[1] = seen ? 1u : 0u;
    }
}

}  // namespace

cudaError_t launch_wait_timeout_probe(uint64_t limit_ns, int code, uint32_t *observed_dev, cudaStream_t stream) {
    wait_timeout_probe_kernel<<<1, 64, 0, stream>>>(limit_ns, code, observed_dev);
    return cudaGetLastError();
}

// Two groups of 128 vectors per CTA (one CTA per SM) when that leaves few rows of the last CTA row
// empty; otherwise one group (two CTAs per SM).
static int tc_vector_groups(int32_t m) {
    const int32_t rest = m % (2 * kTcVectors);
    return (m >= 2 * kTcVectors && (rest == 0 || rest > kTcVectors + kTcVectors / 2 || m >= 16 * kTcVectors)) ? 2 : 1;
}

int32_t project_tc_max_group(int32_t m) { return tc_vector_groups(m) == 2 ? kTcMaxN : 32; }

bool project_tc_applies(int32_t n_group, int32_t m) {
    // enough machines for the tensor core to pay (with five or more the multiply-adds of the scalar kernel cost
    // more issue slots than this kernel's staging and hand-over), enough vectors to fill most of the 128 rows
    // of the last CTA row
    return n_group >= kTcMinMachines && n_group <= project_tc_max_group(m) && m >= 96 &&
           (m % kTcVectors == 0 || m % kTcVectors >= 64 || m >= 1024);
}

template <int NT, int VG>
static size_t tc_smem_bytes(bool bf16) {
    return bf16 ? TcShape<NT, true, VG>::kSmemBytes : TcShape<NT, false, VG>::kSmemBytes;
}

void fill_project_tc_plan(ProjectPlan &p, int32_t n_group, int32_t m, int64_t d, int dtype, int sm_count) {
    const int vg = tc_vector_groups(m);
    p.mma = 2;
    p.nb = n_group > 32 ? 64 : n_group > 16 ? 32 : 16;     // N of the instruction
    p.jt = 4 * vg;                     // producer thread = (lane, warp): 4 or 8 vectors x 1 block per stage
    p.uq = 1;
    p.tile_q = kTcTileBlocks;
    p.tj = 32;
    p.tq = kTcWarps;
    p.grid_y = (m + vg * kTcVectors - 1) / (vg * kTcVectors);
    p.tiles = (d + 4 * (int64_t)kTcTileBlocks - 1) / (4 * (int64_t)kTcTileBlocks);
    const bool bf16 = dtype == 1;
    if (vg == 2) p.smem = p.nb == 64 ? tc_smem_bytes<64, 2>(bf16) : p.nb == 32 ? tc_smem_bytes<32, 2>(bf16) : tc_smem_bytes<16, 2>(bf16);
    else p.smem = p.nb == 32 ? tc_smem_bytes<32, 1>(bf16) : tc_smem_bytes<16, 1>(bf16);
    int64_t gx = (int64_t)sm_count * (vg == 2 ? 1 : 2) / p.grid_y;
    if (gx < 1) gx = 1;
    if (gx > p.tiles) gx = p.tiles;
    p.grid_x = (int)gx;
}

cudaError_t launch_project_tc(const ProjectPlan &plan, const RoundKeys &keys, uint32_t t, const void *G, int dtype,
                              int32_t n, int64_t ldg, int64_t d, int32_t m, uint64_t q_base, float *partial,
                              cudaStream_t stream) {
    if (q_base % kTcTileBlocks != 0 || n > plan.nb || (plan.nb != 16 && plan.nb != 32 && plan.nb != 64) ||
        (plan.jt != 4 && plan.jt != 8) || (plan.nb == 64 && plan.jt != 8))
        return cudaErrorInvalidValue;
    TcArgs a{};
    a.G = G;
    a.ldg = ldg;
    a.d = d;
    a.tiles = plan.tiles;
    a.q_base = q_base;
    a.partial = partial;
    a.n = n;
    a.m = m;
    const size_t es = dtype == 1 ? 2 : 4;
    a.aligned = ((reinterpret_cast<uintptr_t>(G) % 16) == 0 && ((size_t)ldg * es) % 16 == 0) ? 1 : 0;
    a.t = t;
    a.keys = keys;
    dim3 grid(plan.grid_x, plan.grid_y);
    auto go = [&](auto kernel) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem);
        if (e != cudaSuccess) return e;
        kernel<<<grid, kTcThreads, plan.smem, stream>>>(a);
        return cudaGetLastError();
    };
    auto pick = [&](auto nt, auto vg) {
        constexpr int NT = decltype(nt)::value, VG = decltype(vg)::value;
        if (dtype == 1) return go(project_tc_kernel<__nv_bfloat16, NT, VG>);
        return go(project_tc_kernel<float, NT, VG>);
    };
    using I16 = std::integral_constant<int, 16>;
    using I32 = std::integral_constant<int, 32>;
    using I1 = std::integral_constant<int, 1>;
    using I2 = std::integral_constant<int, 2>;
    using I64 = std::integral_constant<int, 64>;
    if (plan.jt == 8) return plan.nb == 64 ? pick(I64{}, I2{}) : plan.nb == 32 ? pick(I32{}, I2{}) : pick(I16{}, I2{});
    return plan.nb == 32 ? pick(I32{}, I1{}) : pick(I16{}, I1{});
}

cudaError_t project_tc_take_status(int *status) {
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return e;
    e = cudaMemcpyFromSymbol(status, g_tc_status, sizeof(int));
    if (e != cudaSuccess) return e;
    const int zero = 0;
    return cudaMemcpyToSymbol(g_tc_status, &zero, sizeof(int));
}

}  // namespace core
