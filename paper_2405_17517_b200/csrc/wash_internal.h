// Internal interface between the C ABI (wash_api.cu) and the kernel launchers.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace wash {

constexpr int kMaxN = 64;          // largest population (WASH_MAX_N)
constexpr int kTileShift = 8;      // lookup tile = 256 groups = 1024 coordinates
constexpr int kDtypeF32 = 0, kDtypeBF16 = 1, kDtypeNone = -1;
constexpr int kLayoutNP = 0, kLayoutPN = 1;
constexpr int kModeStream = 0, kModeSparse = 1;

// One row of a stack is cut into groups of 4 consecutive elements; a group never
// straddles two tensors because tensors start on multiples of 8 elements.
struct SegEntry {
    uint32_t group_begin;   // first group of the segment within a row
    uint32_t group_end;     // one past its last group (padding groups included)
    uint32_t tensor_id;     // RNG tensor index
    uint32_t cgroup_begin;  // (first coordinate's index within its tensor) / 4
    uint32_t numel;         // coordinates in the segment
    uint32_t reserved;
    uint64_t thr;           // floor(p * 2^32): coordinate selected iff word < thr
};
static_assert(sizeof(SegEntry) == 32, "SegEntry must stay 32 bytes");

// Statistics are gathered in kStatSlots partial sums before they reach the caller's two
// counters: per-block atomics on one address were measured to cost about 1 ns each and
// to dominate the kernel once most blocks have a selected coordinate.
constexpr int kStatSlots = 256;
struct StatSlot {
    unsigned long long selected, moved, blocks, reserved;
};

struct PopView {
    int N;
    int layout;
    long long padded_P;           // elements per model row
    uint32_t n_groups;            // padded_P / 4
    int n_seg;
    const SegEntry *seg;          // device, n_seg entries
    const uint32_t *tile_first;   // device, segment of the first group of every tile
};

// Philox's key schedule: round r of the ten uses (k[2r], k[2r+1]) = (seed_lo + r W0, seed_hi + r W1)
// with the two Weyl constants.  It depends on the seed only, so the host computes it once per
// launch and a round's key reaches the kernel as an operand instead of two additions.
struct PhiloxKeys {
    uint32_t k[20];
};
inline PhiloxKeys philox_keys(uint64_t seed)
{
    PhiloxKeys keys;
    uint32_t k0 = static_cast<uint32_t>(seed), k1 = static_cast<uint32_t>(seed >> 32);
    for (int r = 0; r < 10; ++r, k0 += 0x9E3779B9u, k1 += 0xBB67AE85u) {
        keys.k[2 * r] = k0;
        keys.k[2 * r + 1] = k1;
    }
    return keys;
}

// Distance to the consensus gathered inside the streaming shuffle: up to kMaxSqRanges ranges of
// segments, per range and model a binary64 sum, gathered in kSqSlots partial copies (atomics on
// one address per model would serialise) that sq_flush_kernel adds into the caller's array.
constexpr int kMaxSqRanges = 8;
constexpr int kSqSlots = 64;
struct SqArgs {
    double *slots = nullptr;                // device: [kSqSlots][n_ranges][N], zero between launches; nullptr = statistic off
    int n_ranges = 0;
    double inv_n = 0.0;                     // 1 / N
    uint32_t seg_bound[kMaxSqRanges + 1];   // range r = segments seg_bound[r] .. seg_bound[r+1]-1
};

struct ShuffleArgs {
    PopView pop;
    void *a;                      // first stack (device)
    void *b;                      // second stack or nullptr
    uint32_t group_lo, group_hi;  // groups of a row to process (whole row: 0 .. n_groups)
    PhiloxKeys keys;              // from the seed
    uint32_t step_lo, step_hi8;   // step & 0xFFFFFFFF, (step >> 32) << 8
    unsigned long long *stats;    // device-accessible {selected, moved} or nullptr
    StatSlot *stat_slots;         // device, kStatSlots zeroed entries (left zeroed by every launch), or nullptr
    uint32_t *status;             // device status word
    SqArgs sq;                    // consensus distance of the first stack (streaming kernel only)
    uint32_t pn_pad = 0;          // streaming kernel, [P][N]: elements of padding after a group in the shared-memory image (0 or 4)
    bool early = false;           // streaming kernel: the flavour that draws permutations while the copies are in flight
    float expected_share = 0.f;   // share of the coordinates the call's probabilities select, in expectation (sizes the sparse kernel's grid)
};

struct ReduceArgs {
    PopView pop;
    void *stack;                  // device stack (read; written by EMA / papa_all)
    void *out;                    // average row (device) or nullptr
    float alpha, one_minus_alpha;
    uint32_t group_lo, group_hi;  // range of groups to process
    double *sq_out;               // consensus: N doubles (device) or nullptr
    uint32_t *status;
};

// One model per device (wash_exchange_*): the row is one model of a population of pop.N.
constexpr int kExchangeTileGroups = 128;   // a warp tile (wash_warp_tiles.cuh): 32 lanes x 4 groups = 512 coordinates
constexpr int kExchangeWarps = 8;          // warps per block of the exchange kernels
#ifndef WASH_EXCHANGE_BLOCKS_PER_SM
#define WASH_EXCHANGE_BLOCKS_PER_SM 4
#endif
constexpr int kExchangeBlocksPerSm = WASH_EXCHANGE_BLOCKS_PER_SM;   // grid of the exchange kernels = this many blocks per SM (what the plan kernel fits)
struct ExchangeArgs {
    PopView pop;
    int self;                     // this worker's index in the population
    uint32_t n_wtiles;            // ceil(n_groups / kExchangeTileGroups)
    uint32_t n_blocks;            // grid of all three kernels; its warps share the warp tiles evenly, in order
    PhiloxKeys keys;
    uint32_t step_lo, step_hi8;
    uint32_t *mask;               // [n_wtiles * 32] a word per lane = its four groups' bytes; low nibble of a byte:
                                  // selected coordinates, high nibble: those this worker receives
    uint32_t *warp_total;         // [n_blocks * kExchangeWarps][N + 1]: column n = slots of worker n's buffer the
                                  // warp's range takes; column N = selected coordinates
    uint32_t *block_total;        // [n_blocks][N + 1] the same per block
    void *row[2];                 // this worker's model: parameters, optimizer state (nullptr: absent)
    int dtype[2];
    void *const *staging[2];      // per stack: device array of N pointers, entry n = worker n's staging buffer
    long long capacity[2];        // elements per staging buffer
    unsigned long long *stats;    // {selected, received} or nullptr
    uint32_t *status;
};
cudaError_t launch_exchange_plan(const ExchangeArgs &args, cudaStream_t stream);
cudaError_t launch_exchange_send(const ExchangeArgs &args, cudaStream_t stream);
cudaError_t launch_exchange_receive(const ExchangeArgs &args, cudaStream_t stream);

enum ReduceOp { kOpEma = 0, kOpAverage = 1, kOpPapaAll = 2, kOpConsensus = 3 };

// The resident-warp streaming kernel takes groups (all models, both stacks) of up to 48 bytes -- fp32 N = 2, 3;
// bf16 N <= 6 -- when at most 30 % of the coordinates are expected to be selected.  Measured on 2^27 coordinates
// against the one-trip kernel: 32 bytes 0.73-0.93 of its time, 48 bytes 0.89-0.98, 64 bytes 0.97-1.12.
constexpr size_t kLoopMaxGroupBytes = 48;
constexpr float kLoopMaxShare = 0.3f;
// Groups of 49 to 64 bytes go to it only for an expected selection between 0.7 % and 5 %: measured at 1 % and 3 %
// it takes 0.89-0.97 of the one-trip kernel's time (both layouts), at 0.3 % 1.01-1.03, at 10 % 0.93 in [P][N] but 1.20 in [N][P].
constexpr size_t kLoopWideGroupBytes = 64;
constexpr float kLoopWideShareLo = 0.007f, kLoopWideShareHi = 0.05f;

struct LaunchShape {
    int threads;         // 0 = default
    int blocks_per_sm;   // <= 0: one group per thread; > 0: persistent grid, that many blocks per SM
    int sm_count;
};

// Each returns cudaSuccess or the launch error; *supported = false (and no launch) if
// the library has no kernel for the combination.
cudaError_t launch_shuffle(const ShuffleArgs &args, int a_dtype, int b_dtype, int mode,
                           const LaunchShape &shape, cudaStream_t stream, bool *supported);
cudaError_t launch_reduce(const ReduceArgs &args, int op, int dtype, int out_dtype,
                          const LaunchShape &shape, cudaStream_t stream, bool *supported);

// adds the slots' sums into out[n_ranges][N] and zeroes the slots
cudaError_t launch_sq_flush(const SqArgs &sq, int N, double *out, cudaStream_t stream);

cudaError_t launch_philox_probe(unsigned long long n_blocks, uint64_t seed, uint32_t *checksum, cudaStream_t stream);

void count_launch();

}  // namespace wash
