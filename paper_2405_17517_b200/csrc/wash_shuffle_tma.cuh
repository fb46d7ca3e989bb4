// Streaming shuffle with the stack staged through shared memory by the bulk-copy
// engine (TMA, cp.async.bulk) instead of through registers.
//
// Why: the register-resident kernel keeps N (or 2N) vectors per thread in flight and is
// limited by how many such threads fit on an SM (measured: 24 warps, ~120 KB in flight
// per SM, 85 % of the bandwidth a pure read reaches).  Measured outcome on B200: every
// 1-D bulk copy costs its CTA about 85 ns whatever its size, so with rows of a few KiB
// this kernel reaches 76-80 % of the measured copy bandwidth on the ResNet populations
// and does not beat the register kernel (83-92 %); it is kept as a selectable mode.  Here the producer warps of a CTA
// stream tiles of the stack into a ring of shared-memory stages with bulk asynchronous
// copies that complete on mbarriers; ~200 KB per SM are in flight with no register
// cost, and the consumer warps spend their time on the Philox mask, which needs no data
// at all.  A consumer touches a stage only for a selected coordinate (it then reads the
// N values from shared memory and writes the moved ones to global memory); a warp hands
// a stage back as soon as it has drawn the tile's mask and served its selected lanes,
// whether or not the tile has landed -- the producers wait for the landing themselves
// before they reuse the stage.  N is a run-time value: one instantiation serves every population size.
//
// Tile = G consecutive groups (G = threads of one consumer team).  [N][P]: one bulk copy
// per model row and stack (G*16 bytes of fp32).  [P][N]: the tile's G*4N elements are
// contiguous, one copy per stack.  Every copy starts on a 16-byte boundary and has a
// size that is a multiple of 16 bytes (rows start on multiples of 8 elements, a group
// is 16 or 8 bytes, G is a multiple of 32).
//
// All waits are bounded: a wait that exceeds kWaitLimitCycles sets bit 1 of the status word
// and an abort flag that every loop checks; the producer then still waits (bounded) for
// the copies it has issued before the CTA returns.
#pragma once
#include "wash_device.cuh"
#include "wash_launch.cuh"

namespace wash {

constexpr long long kWaitLimitCycles = 4000000000ll;   // about 2 s of SM clock
constexpr int kMaxStages = 12;
constexpr int kHeaderBytes = 512;   // three barriers per stage and the abort flag
constexpr int kProducerWarps = 1;
constexpr int kCtasPerSm = 3;
constexpr int kPieceBytes = 4096;   // largest single bulk copy

struct ShuffleTmaArgs {
    ShuffleArgs s;
    uint32_t n_tiles;        // ceil(n_groups / G)
    int G;                   // groups per tile = threads per consumer team
    int teams;               // consumer teams per CTA (tile i of a CTA goes to team i % teams); divides stages
    int stages;
    uint32_t stage_bytes;    // bytes of one stage (both stacks)
    uint32_t b_offset;       // byte offset of the second stack inside a stage
    uint32_t seg_smem_bytes; // bytes reserved for a shared-memory copy of the segment table (0: read it from global)
};

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Waits for the phase of parity `parity` to complete.  Returns false if the CTA is
// aborting or the wait ran out of time (then it sets the abort flag and the status bit).
// Time is measured with the SM's cycle counter, read only every 1024 polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t *status, uint32_t site = 0)
{
    if (mbar_try_wait(bar, parity)) return true;
    long long t0 = 0;
    for (uint32_t polls = 1;; ++polls) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((polls & 1023u) == 0) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            if (now - t0 > kWaitLimitCycles) {
                *abort_flag = 1;
                if (status) atomicOr(status, 2u | site);
                return false;
            }
        }
    }
}
// global -> shared bulk copy that reports its bytes to an mbarrier of this CTA
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// pi for coordinate i in a column of bytes: s_perm[n * stride]
static __device__ __noinline__ void draw_permutation_u8(uint8_t *s_perm, int stride, int n_models, uint32_t i,
                                                        uint32_t tensor, uint32_t step_lo, uint32_t step_hi8,
                                                        const PhiloxKeys &keys)
{
    for (int n = 0; n < n_models; ++n) s_perm[n * stride] = static_cast<uint8_t>(n);
    Philox4 w{0, 0, 0, 0};
    for (int k = n_models - 1, m = 0; k >= 1; --k, ++m) {
        if ((m & 3) == 0) w = philox4x32_10(i, tensor, step_lo, step_hi8 | (1u + (static_cast<uint32_t>(m) >> 2)), keys);
        const uint32_t r = w.x;
        w.x = w.y; w.y = w.z; w.z = w.w;
        const uint32_t j = __umulhi(r, static_cast<uint32_t>(k + 1));
        const uint8_t pk = s_perm[k * stride], pj = s_perm[j * stride];
        s_perm[k * stride] = pj;
        s_perm[j * stride] = pk;
    }
}

// raw bits of (model n, coordinate c) of the tile's group j, read from a stage
template <class T, int LAYOUT>
__device__ __forceinline__ uint32_t stage_value(const unsigned char *stage, int G, int n_models, int n, int j, int c)
{
    const uint32_t elem = LAYOUT == kLayoutNP ? (static_cast<uint32_t>(n) * G + j) * 4u + c
                                              : (static_cast<uint32_t>(j) * 4u + c) * n_models + n;
    if (T::kBytes == 4) return reinterpret_cast<const uint32_t *>(stage)[elem];
    return reinterpret_cast<const uint16_t *>(stage)[elem];
}

template <class TA, class TB, int LAYOUT>
__global__ void __launch_bounds__(32 * kProducerWarps + 512) shuffle_tma_kernel(const __grid_constant__ ShuffleTmaArgs a)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    constexpr bool kHasB = TB::kCode != kDtypeNone;
    // shared memory: [0,512) barriers + abort flag | stages | permutation columns | segment table
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_raw);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_raw + 8 * 3 * kMaxStages);
    unsigned char *stage0 = smem_raw + kHeaderBytes;
    const int S = a.stages, G = a.G, n_models = a.s.pop.N;
    const int consumers = G * a.teams;
    uint8_t *perm_base = stage0 + static_cast<size_t>(S) * a.stage_bytes;
    // optional copy of the segment table, so that the lookup costs no global round trip
    const SegEntry *seg = a.s.pop.seg;
    if (a.seg_smem_bytes) {
        uint4 *dst = reinterpret_cast<uint4 *>(perm_base + ((static_cast<size_t>(n_models) * consumers + 15) & ~static_cast<size_t>(15)));
        const uint4 *src = reinterpret_cast<const uint4 *>(a.s.pop.seg);
        for (int k = threadIdx.x; k < a.s.pop.n_seg * 2; k += blockDim.x) dst[k] = __ldg(src + k);
        seg = reinterpret_cast<const SegEntry *>(dst);
    }
    // per stage: full (the tile's bytes have landed), empty (every consumer warp has let go of
    // the stage), issued (the producers have started the tile's copies)
    const uint32_t full0 = smem_addr(bars), empty0 = smem_addr(bars + kMaxStages), issued0 = smem_addr(bars + 2 * kMaxStages);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int warps_per_team = G >> 5;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full0 + 8 * s, kProducerWarps);
            mbar_init(empty0 + 8 * s, warps_per_team);
            mbar_init(issued0 + 8 * s, kProducerWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // tiles of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ...
    const uint32_t my_tiles = blockIdx.x < a.n_tiles ? (a.n_tiles - 1 - blockIdx.x) / gridDim.x + 1 : 0;
    const uint32_t vec_a = TA::kBytes * 4, vec_b = kHasB ? TB::kBytes * 4 : 0;

    if (warp < kProducerWarps) {
        // ---------------- producers ----------------
        // A tile is a list of contiguous regions ([N][P]: one per model row and stack;
        // [P][N]: one per stack), cut into pieces of at most kPieceBytes.  Piece q goes to
        // a producer thread, warps taking turns: each bulk copy occupies its issuing warp for some tens of
        // nanoseconds, so the pieces are spread over several warps.  Lane 0 of every producer
        // warp announces the warp's bytes with its arrival (arrive.expect_tx) before the
        // warp issues its copies, so a stage's "full" barrier counts kProducerWarps arrivals.
        const int regions_a = LAYOUT == kLayoutNP ? n_models : 1;
        const int regions_b = kHasB ? regions_a : 0;
        uint32_t issued = 0;
        for (uint32_t i = 0; i < my_tiles; ++i) {
            const int s = static_cast<int>(i % S);
            // lane 0 waits for the stage to be free; the answer is made warp-uniform
            // (the stage's previous tile must have landed, so that the barrier's byte count
            // is settled, and every consumer warp must have let go of it)
            int go = 1;
            if (lane == 0) {
                if (i >= static_cast<uint32_t>(S))
                    go = (mbar_wait(full0 + 8 * s, ((i / S) - 1) & 1u, abort_flag, a.s.status, 16u) &&
                          mbar_wait(empty0 + 8 * s, ((i / S) - 1) & 1u, abort_flag, a.s.status, 32u)) ? 1 : 0;
                else go = *abort_flag ? 0 : 1;
            }
            go = __shfl_sync(0xFFFFFFFFu, go, 0);
            if (!go) break;
            const uint64_t tile = blockIdx.x + static_cast<uint64_t>(i) * gridDim.x;
            const uint64_t g0 = tile * G;
            const uint32_t groups = static_cast<uint32_t>(min(static_cast<uint64_t>(G), a.s.pop.n_groups - g0));
            const uint32_t dst = smem_addr(stage0 + static_cast<size_t>(s) * a.stage_bytes);
            const uint32_t bar = full0 + 8 * s;
            // bytes of one region of each stack, and how many pieces that makes
            const uint32_t bytes_a = groups * vec_a * (LAYOUT == kLayoutNP ? 1 : n_models);
            const uint32_t bytes_b = groups * vec_b * (LAYOUT == kLayoutNP ? 1 : n_models);
            const uint32_t pieces_a = (bytes_a + kPieceBytes - 1) / kPieceBytes;
            const uint32_t pieces_b = kHasB ? (bytes_b + kPieceBytes - 1) / kPieceBytes : 0;
            const uint32_t total = regions_a * pieces_a + regions_b * pieces_b;
            // this warp's share of the bytes, announced by lane 0 together with its arrival
            uint32_t my_bytes = 0;
            for (uint32_t q = lane * kProducerWarps + warp; q < total; q += 32 * kProducerWarps) {
                const bool in_a = q < regions_a * pieces_a;
                const uint32_t qq = in_a ? q : q - regions_a * pieces_a;
                const uint32_t per = in_a ? pieces_a : pieces_b;
                const uint32_t off = (qq % per) * kPieceBytes;
                my_bytes += min(static_cast<uint32_t>(kPieceBytes), (in_a ? bytes_a : bytes_b) - off);
            }
            my_bytes = __reduce_add_sync(0xFFFFFFFFu, my_bytes);
            if (lane == 0) mbar_arrive_expect_tx(bar, my_bytes);
            __syncwarp();
            for (uint32_t q = lane * kProducerWarps + warp; q < total; q += 32 * kProducerWarps) {   // neighbouring pieces go to different warps
                const bool in_a = q < regions_a * pieces_a;
                const uint32_t qq = in_a ? q : q - regions_a * pieces_a;
                const uint32_t per = in_a ? pieces_a : pieces_b;
                const uint32_t region = qq / per, off = (qq - region * per) * kPieceBytes;
                const uint32_t bytes = min(static_cast<uint32_t>(kPieceBytes), (in_a ? bytes_a : bytes_b) - off);
                const int eb = in_a ? TA::kBytes : (kHasB ? TB::kBytes : 1);
                // first element of the region in the stack, and its place in the stage
                const long long elem0 = LAYOUT == kLayoutNP ? static_cast<long long>(region) * a.s.pop.padded_P + 4ll * g0
                                                            : 4ll * g0 * n_models;
                const char *src = static_cast<const char *>(in_a ? a.s.a : a.s.b) + elem0 * eb + off;
                const uint32_t region_dst = (in_a ? 0u : a.b_offset) + (LAYOUT == kLayoutNP ? region * G * (in_a ? vec_a : vec_b) : 0u);
                bulk_load(dst + region_dst + off, src, bytes, bar);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(issued0 + 8 * s);
            issued = i + 1;
        }
        // Do not leave while copies into this CTA's shared memory may be in flight: in
        // the normal case these phases completed long ago and the checks return at once.
        if (lane == 0) {
            const uint32_t first = issued > static_cast<uint32_t>(S) ? issued - S : 0;
            for (uint32_t i = first; i < issued; ++i) {
                const uint32_t bar = full0 + 8 * (i % S);
                const long long t0 = clock64();
                while (!mbar_try_wait(bar, (i / S) & 1u))
                    if (clock64() - t0 > kWaitLimitCycles) { if (a.s.status) atomicOr(a.s.status, 4u); break; }
            }
        }
        return;
    }

    // ---------------- consumers ----------------
    const int ct = threadIdx.x - 32 * kProducerWarps;   // consumer thread index
    if (ct >= consumers) return;
    const int team = ct / G, j = ct - team * G;      // j: group of the tile this thread owns
    uint8_t *s_perm = perm_base + ct;                // column [n][consumers]
    uint32_t selected = 0, moved = 0;
    // this thread's groups come in increasing order: the segment cursor only moves forward
    uint32_t cursor = 0;
    {
        const uint64_t g_first = (blockIdx.x + static_cast<uint64_t>(team) * gridDim.x) * G + j;
        if (static_cast<uint32_t>(team) < my_tiles && g_first < a.s.pop.n_groups) cursor = __ldg(a.s.pop.tile_first + (g_first >> kTileShift));
    }
    for (uint32_t i = team; i < my_tiles; i += a.teams) {
        if (*abort_flag) break;
        const int s = static_cast<int>(i % S);
        const uint32_t parity = (i / S) & 1u;
        const uint32_t full = full0 + 8 * s;
        const uint64_t tile = blockIdx.x + static_cast<uint64_t>(i) * gridDim.x;
        const uint64_t g = tile * G + j;
        uint32_t sel = 0;
        GroupInfo gi{0, 0, 0, 0};
        if (g < a.s.pop.n_groups) {
            gi = find_group_forward(seg, a.s.pop.n_seg, cursor, static_cast<uint32_t>(g), a.s.status);
            if (gi.thr != 0 && gi.valid != 0) {
                const Philox4 w = philox4x32_10(gi.cgroup, gi.tensor_id, a.s.step_lo, a.s.step_hi8, a.s.keys);
                sel |= (static_cast<uint64_t>(w.x) < gi.thr && gi.valid > 0) ? 1u : 0u;
                sel |= (static_cast<uint64_t>(w.y) < gi.thr && gi.valid > 1) ? 2u : 0u;
                sel |= (static_cast<uint64_t>(w.z) < gi.thr && gi.valid > 2) ? 4u : 0u;
                sel |= (static_cast<uint64_t>(w.w) < gi.thr && gi.valid > 3) ? 8u : 0u;
            }
        }
        // Only a thread with a selected coordinate needs the tile's data.  Its warp may have
        // released the stage's previous tile before that tile had landed, and a parity wait
        // cannot tell "previous phase still open" from "this phase already over".  So it
        // first waits until the producers have issued this tile -- which they only do once
        // the previous one has landed -- and then for this tile's bytes.
        const uint32_t k = i / S;
        if (sel != 0 && mbar_wait(issued0 + 8 * s, parity, abort_flag, a.s.status, 64u) &&
            mbar_wait(full, parity, abort_flag, a.s.status, 128u)) {
            const unsigned char *stage = stage0 + static_cast<size_t>(s) * a.stage_bytes;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                if (!((sel >> c) & 1u)) continue;
                draw_permutation_u8(s_perm, consumers, n_models, 4u * gi.cgroup + c, gi.tensor_id, a.s.step_lo, a.s.step_hi8, a.s.keys);
                const long long e = 4ll * static_cast<long long>(g) + c;
                for (int n = 0; n < n_models; ++n) {
                    const int src = s_perm[n * consumers];
                    if (src == n) continue;
                    TA::store_elem(a.s.a, elem_index<LAYOUT>(a.s.pop, n, e), stage_value<TA, LAYOUT>(stage, G, n_models, src, j, c));
                    if constexpr (kHasB)
                        TB::store_elem(a.s.b, elem_index<LAYOUT>(a.s.pop, n, e), stage_value<TB, LAYOUT>(stage + a.b_offset, G, n_models, src, j, c));
                    ++moved;
                }
                ++selected;
            }
        }
        __syncwarp();
        // Release the stage for this tile.  An arrival counts toward the barrier's current
        // phase, so the previous phase (every warp's release of the stage's previous tile)
        // has to be over first.  The warp does not wait for the tile's data: a stage whose
        // tile nobody needs is handed back before it has even landed, and the producers
        // check the landing themselves.
        // Nor may the consumers get more than one phase ahead of the producers (a parity wait
        // can only tell two neighbouring phases apart): the release also waits until the
        // producers have issued this tile, which they do long before it lands.
        if (lane == 0 && (k == 0 || mbar_wait(empty0 + 8 * s, parity ^ 1u, abort_flag, a.s.status, 256u)) &&
            mbar_wait(issued0 + 8 * s, parity, abort_flag, a.s.status, 512u))
            mbar_arrive(empty0 + 8 * s);
        __syncwarp();
    }
    if (a.s.stats) {
        selected = __reduce_add_sync(0xFFFFFFFFu, selected);
        moved = __reduce_add_sync(0xFFFFFFFFu, moved);
        if (lane == 0 && selected) {
            atomicAdd(a.s.stats, static_cast<unsigned long long>(selected));
            atomicAdd(a.s.stats + 1, static_cast<unsigned long long>(moved));
        }
    }
}

// Picks tile size, stage count and grid for the population and launches.
template <class TA, class TB>
cudaError_t launch_shuffle_tma_typed(const ShuffleArgs &args, const LaunchShape &shape, cudaStream_t stream)
{
    constexpr bool kHasB = TB::kCode != kDtypeNone;
    const int N = args.pop.N;
    const uint32_t group_bytes = static_cast<uint32_t>(N) * (TA::kBytes * 4 + (kHasB ? TB::kBytes * 4 : 0));
    // Each bulk copy costs its CTA a fixed ~85 ns whatever its size (measured), so one CTA
    // cannot keep an SM's share of HBM busy with copies of a few KiB: aim for kCtasPerSm
    // CTAs per SM, each with its own ring, and fall back to fewer when a population's
    // stages are too large for that.
    int ctas = kCtasPerSm;
    ShuffleTmaArgs t;
    t.s = args;
    int stages = 0;
    size_t perm_bytes = 0;
    const size_t seg_bytes = sizeof(SegEntry) * static_cast<size_t>(args.pop.n_seg);
    t.seg_smem_bytes = seg_bytes <= 16 * 1024 ? static_cast<uint32_t>(seg_bytes) : 0;
    for (; ctas >= 1; --ctas) {
        const size_t budget = 200 * 1024 / ctas;
        int G = 256;
        if (shape.threads == 128 || shape.threads == 64 || shape.threads == 32) G = shape.threads;
        while (G > 32 && 2ull * G * group_bytes + static_cast<size_t>(N) * G + t.seg_smem_bytes > budget) G >>= 1;
        t.G = G;
        t.teams = 1;
        if (shape.blocks_per_sm > 0) t.teams = shape.blocks_per_sm;   // tuning: consumer teams per CTA
        if (t.teams * G > 512) t.teams = 512 / G;
        t.stage_bytes = static_cast<uint32_t>(G) * group_bytes;
        t.b_offset = static_cast<uint32_t>(G) * N * TA::kBytes * 4;
        perm_bytes = (static_cast<size_t>(N) * G * t.teams + 15) & ~static_cast<size_t>(15);   // sized for the most teams considered
        if (perm_bytes + t.seg_smem_bytes >= budget) continue;
        stages = static_cast<int>((budget - perm_bytes - t.seg_smem_bytes) / t.stage_bytes);
        if (stages > kMaxStages) stages = kMaxStages;
        // A stage must always be consumed by the same team: a waiter has to see every
        // phase of the barriers it waits on.
        while (t.teams > 1 && stages / t.teams * t.teams < 2) t.teams >>= 1;
        stages = stages / t.teams * t.teams;
        if (stages >= 2) break;
    }
    if (stages < 2) return cudaErrorInvalidConfiguration;
    const int G = t.G;
    t.stages = stages;
    t.n_tiles = (args.pop.n_groups + G - 1) / G;
    const size_t smem = kHeaderBytes + static_cast<size_t>(stages) * t.stage_bytes + perm_bytes + t.seg_smem_bytes;
    const int threads = 32 * kProducerWarps + G * t.teams;
    auto kernel = args.pop.layout == kLayoutNP ? shuffle_tma_kernel<TA, TB, kLayoutNP> : shuffle_tma_kernel<TA, TB, kLayoutPN>;
    KernelFit fit;
    cudaError_t err = kernel_fit(reinterpret_cast<const void *>(kernel), threads, smem, &fit);
    if (err != cudaSuccess) return err;
    if (fit.occupancy < 1) return cudaErrorLaunchOutOfResources;
    uint64_t grid = static_cast<uint64_t>(shape.sm_count > 0 ? shape.sm_count : 148) * fit.occupancy;
    if (grid > t.n_tiles) grid = t.n_tiles;
    if (grid == 0) return cudaSuccess;
    kernel<<<static_cast<unsigned>(grid), threads, smem, stream>>>(t);
    count_launch();
    return cudaGetLastError();
}

inline cudaError_t launch_shuffle_tma(const ShuffleArgs &args, int a_dtype, int b_dtype, const LaunchShape &shape,
                                      cudaStream_t stream, bool *supported)
{
    *supported = true;
    if (a_dtype == kDtypeF32 && b_dtype == kDtypeNone) return launch_shuffle_tma_typed<F32, NoStack>(args, shape, stream);
    if (a_dtype == kDtypeBF16 && b_dtype == kDtypeNone) return launch_shuffle_tma_typed<BF16, NoStack>(args, shape, stream);
    if (a_dtype == kDtypeF32 && b_dtype == kDtypeF32) return launch_shuffle_tma_typed<F32, F32>(args, shape, stream);
    if (a_dtype == kDtypeBF16 && b_dtype == kDtypeF32) return launch_shuffle_tma_typed<BF16, F32>(args, shape, stream);
    if (a_dtype == kDtypeBF16 && b_dtype == kDtypeBF16) return launch_shuffle_tma_typed<BF16, BF16>(args, shape, stream);
    if (a_dtype == kDtypeF32 && b_dtype == kDtypeBF16) return launch_shuffle_tma_typed<F32, BF16>(args, shape, stream);
    *supported = false;
    return cudaSuccess;
}

}  // namespace wash
