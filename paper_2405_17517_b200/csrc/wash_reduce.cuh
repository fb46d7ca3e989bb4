// The dense comparison operators, each one fused pass over the stack:
//   kOpEma       PAPA's EMA, Eq. 1:  x_n <- alpha x_n + (1 - alpha) m
//   kOpAverage   the averaged model (output of Algorithm 1): out <- m
//   kOpPapaAll   PAPA-all / DART: x_n <- m
//   kOpConsensus squared distances to the consensus (Eq. 2 / Eq. 5 / Fig. 2)
// with m = (((x_0 + x_1) + x_2) + ...)/N in binary32, each operation rounded once
// (explicit _rn intrinsics: the compiler may neither fuse nor reorder them).
//
// A thread owns one group of 4 coordinates for all N models, as in the shuffle.
#pragma once
#include "wash_device.cuh"
#include "wash_launch.cuh"

namespace wash {

template <int N, class T, class TOUT, int LAYOUT, int OP>
__global__ void __launch_bounds__(256) reduce_kernel(const __grid_constant__ ReduceArgs a)
{
    constexpr int kCap = N > 0 ? N : kMaxN;
    const int n_models = N > 0 ? N : a.pop.N;
    const float inv_count = static_cast<float>(n_models);
    double acc[OP == kOpConsensus ? kCap : 1];
    if constexpr (OP == kOpConsensus) {
#pragma unroll
        for (int n = 0; n < kCap; ++n) acc[n] = 0.0;
    }
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    for (uint64_t g = a.group_lo + static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x; g < a.group_hi; g += stride) {
        typename T::vec v[kCap];
        if constexpr (N > 0) {
#pragma unroll
            for (int j = 0; j < N; ++j) v[j] = T::load_group(group_vec_ptr<T, LAYOUT>(a.stack, a.pop, g, j));
        } else {
            for (int j = 0; j < n_models; ++j) v[j] = T::load_group(group_vec_ptr<T, LAYOUT>(a.stack, a.pop, g, j));
        }
        const GroupInfo gi = find_group(a.pop, static_cast<uint32_t>(g), a.status);
        if (gi.valid == 0) continue;

        if constexpr (OP == kOpConsensus) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if (c >= gi.valid) break;
                double sum = 0.0;
#pragma unroll
                for (int n = 0; n < kCap; ++n)
                    if (n < n_models) sum += static_cast<double>(T::to_float(group_value<T, LAYOUT, kCap>(v, n_models, n, c)));
                const double mean = sum / static_cast<double>(n_models);
#pragma unroll
                for (int n = 0; n < kCap; ++n)
                    if (n < n_models) {
                        const double d = static_cast<double>(T::to_float(group_value<T, LAYOUT, kCap>(v, n_models, n, c))) - mean;
                        acc[n] += d * d;
                    }
            }
            continue;
        } else {
            // consensus m of the 4 coordinates, binary32, terms in model order
            float m[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float s = T::to_float(group_value<T, LAYOUT, kCap>(v, n_models, 0, c));
#pragma unroll
                for (int n = 1; n < kCap; ++n)
                    if (n < n_models) s = __fadd_rn(s, T::to_float(group_value<T, LAYOUT, kCap>(v, n_models, n, c)));
                m[c] = __fdiv_rn(s, inv_count);
            }
            if constexpr (OP == kOpAverage) {
                const long long e0 = 4ll * static_cast<long long>(g);
                if (gi.valid == 4) {
                    TOUT::store_group(static_cast<char *>(a.out) + e0 * TOUT::kBytes, TOUT::pack_floats(m[0], m[1], m[2], m[3]));
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if (c < gi.valid) TOUT::store_elem(a.out, e0 + c, TOUT::from_float(m[c]));
                }
            } else {
                // new value of (model n, coordinate c)
                auto updated = [&](int n, int c) -> float {
                    if constexpr (OP == kOpPapaAll) return m[c];
                    const float x = T::to_float(group_value<T, LAYOUT, kCap>(v, n_models, n, c));
                    return __fadd_rn(__fmul_rn(a.alpha, x), __fmul_rn(a.one_minus_alpha, m[c]));
                };
                if (gi.valid == 4) {
#pragma unroll
                    for (int j = 0; j < kCap; ++j) {
                        if (j >= n_models) break;
                        float r[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            // element q of vector j is (model n, coordinate c):
                            const int n = LAYOUT == kLayoutNP ? j : (4 * j + q) % n_models;
                            const int c = LAYOUT == kLayoutNP ? q : (4 * j + q) / n_models;
                            r[q] = updated(n, c);
                        }
                        T::store_group(group_vec_ptr<T, LAYOUT>(a.stack, a.pop, g, j), T::pack_floats(r[0], r[1], r[2], r[3]));
                    }
                } else {
                    const long long e0 = 4ll * static_cast<long long>(g);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        if (c >= gi.valid) break;
#pragma unroll
                        for (int n = 0; n < kCap; ++n)
                            if (n < n_models) T::store_elem(a.stack, elem_index<LAYOUT>(a.pop, n, e0 + c), T::from_float(updated(n, c)));
                    }
                }
            }
        }
    }
    if constexpr (OP == kOpConsensus) {
        // warp sums, then one atomic per warp and model
#pragma unroll
        for (int n = 0; n < kCap; ++n) {
            if (n >= n_models) break;
            double s = acc[n];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) s += __shfl_down_sync(0xFFFFFFFFu, s, off);
            if ((threadIdx.x & 31) == 0 && s != 0.0) atomicAdd(a.sq_out + n, s);
        }
    }
}

template <int N, class T, class TOUT, int OP>
cudaError_t launch_reduce_typed(const ReduceArgs &args, const LaunchShape &shape, cudaStream_t stream)
{
    const uint64_t items = args.group_hi > args.group_lo ? args.group_hi - args.group_lo : 0;
    if (args.pop.layout == kLayoutNP)
        return launch_grid_stride(reduce_kernel<N, T, TOUT, kLayoutNP, OP>, args, items, 0, shape, stream);
    return launch_grid_stride(reduce_kernel<N, T, TOUT, kLayoutPN, OP>, args, items, 0, shape, stream);
}

template <int N>
cudaError_t launch_reduce_n(const ReduceArgs &args, int op, int dtype, int out_dtype, const LaunchShape &shape,
                            cudaStream_t stream, bool *supported)
{
    *supported = true;
    const bool f32 = dtype == kDtypeF32, bf16 = dtype == kDtypeBF16;
    if (!f32 && !bf16) { *supported = false; return cudaSuccess; }
    switch (op) {
    case kOpEma:
        return f32 ? launch_reduce_typed<N, F32, F32, kOpEma>(args, shape, stream)
                   : launch_reduce_typed<N, BF16, BF16, kOpEma>(args, shape, stream);
    case kOpPapaAll:
        return f32 ? launch_reduce_typed<N, F32, F32, kOpPapaAll>(args, shape, stream)
                   : launch_reduce_typed<N, BF16, BF16, kOpPapaAll>(args, shape, stream);
    case kOpConsensus:
        return f32 ? launch_reduce_typed<N, F32, F32, kOpConsensus>(args, shape, stream)
                   : launch_reduce_typed<N, BF16, BF16, kOpConsensus>(args, shape, stream);
    case kOpAverage:
        if (f32 && out_dtype == kDtypeF32) return launch_reduce_typed<N, F32, F32, kOpAverage>(args, shape, stream);
        if (f32 && out_dtype == kDtypeBF16) return launch_reduce_typed<N, F32, BF16, kOpAverage>(args, shape, stream);
        if (bf16 && out_dtype == kDtypeF32) return launch_reduce_typed<N, BF16, F32, kOpAverage>(args, shape, stream);
        if (bf16 && out_dtype == kDtypeBF16) return launch_reduce_typed<N, BF16, BF16, kOpAverage>(args, shape, stream);
        break;
    default:
        break;
    }
    *supported = false;
    return cudaSuccess;
}

}  // namespace wash
