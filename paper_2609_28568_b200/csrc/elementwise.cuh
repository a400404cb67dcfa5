// HBM-bound helper kernels around the GEMMs: activation backward (dz), the stand-alone dbias
// column reduction, and the bounded-wait self-test.
#pragma once
#include "gemm_sm100.cuh"

namespace nb {

__device__ __forceinline__ float silu_bwd(float g)
{
    const float s = __fdividef(1.0f, 1.0f + __expf(-g));
    return s * (1.0f + g * (1.0f - s));
}

// dz = dout * gelu'(pre), 8 bf16 per thread per iteration (128-bit loads and stores).
__global__ void __launch_bounds__(256)
gelu_backward_kernel(uint4 *__restrict__ dz, const uint4 *__restrict__ dout,
                     const uint4 *__restrict__ pre, long long nvec)
{
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < nvec;
         i += stride) {
        const uint4 d = __ldg(dout + i);
        const uint4 x = __ldg(pre + i);
        const uint32_t dv[4] = {d.x, d.y, d.z, d.w};
        const uint32_t xv[4] = {x.x, x.y, x.z, x.w};
        uint32_t o[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float lo = ptx::bf16_lo(dv[k]) * gelu_bwd(ptx::bf16_lo(xv[k]));
            const float hi = ptx::bf16_hi(dv[k]) * gelu_bwd(ptx::bf16_hi(xv[k]));
            o[k] = ptx::pack_bf16x2(lo, hi);
        }
        dz[i] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// SwiGLU backward: dout [BT, H], pre [BT, 2H] = [gate | up]  ->  dz [BT, 2H].
//   dz[:, j] = dout * up * silu'(gate) ; dz[:, H + j] = dout * silu(gate)
__global__ void __launch_bounds__(256)
swiglu_backward_kernel(uint4 *__restrict__ dz, const uint4 *__restrict__ dout,
                       const uint4 *__restrict__ pre, long long BT, int hvec /* H / 8 */)
{
    const long long total = BT * hvec;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += stride) {
        const long long m = i / hvec;
        const int j = static_cast<int>(i - m * hvec);
        const uint4 d = __ldg(dout + i);
        const uint4 g = __ldg(pre + m * 2 * hvec + j);
        const uint4 u = __ldg(pre + m * 2 * hvec + hvec + j);
        const uint32_t dv[4] = {d.x, d.y, d.z, d.w};
        const uint32_t gv[4] = {g.x, g.y, g.z, g.w};
        const uint32_t uv[4] = {u.x, u.y, u.z, u.w};
        uint32_t og[4], ou[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float d0 = ptx::bf16_lo(dv[k]), d1 = ptx::bf16_hi(dv[k]);
            const float g0 = ptx::bf16_lo(gv[k]), g1 = ptx::bf16_hi(gv[k]);
            const float u0 = ptx::bf16_lo(uv[k]), u1 = ptx::bf16_hi(uv[k]);
            og[k] = ptx::pack_bf16x2(d0 * u0 * silu_bwd(g0), d1 * u1 * silu_bwd(g1));
            ou[k] = ptx::pack_bf16x2(d0 * silu_fwd(g0), d1 * silu_fwd(g1));
        }
        dz[m * 2 * hvec + j] = make_uint4(og[0], og[1], og[2], og[3]);
        dz[m * 2 * hvec + hvec + j] = make_uint4(ou[0], ou[1], ou[2], ou[3]);
    }
}

// dbias[o] += sum over a block of rows of dz[m, o].
// A block owns 128 columns and `rows_per_block` rows. Inside a warp, lanes 0..7 hold eight
// 128-bit column vectors (64 columns) and the lane's upper bits select one of four rows, for two
// 64-column halves; rows are summed in registers, then across the four row lanes by shuffles,
// across the eight warps by shared-memory atomics, and across blocks by global atomic adds.
constexpr int kDbiasCols = 128;
constexpr int kDbiasThreads = 256;

__global__ void __launch_bounds__(kDbiasThreads)
dbias_kernel(float *__restrict__ dbias, const __nv_bfloat16 *__restrict__ dz, long long BT, int OC,
             int rows_per_block)
{
    // 512 bytes of shared memory only: small enough to share an SM with a resident GEMM CTA
    __shared__ float part[kDbiasCols];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cv = lane & 7;   // column vector inside a 64-column half
    const int rs = lane >> 3;  // row inside a group of four
    const int col0 = blockIdx.x * kDbiasCols;
    const long long r_begin = static_cast<long long>(blockIdx.y) * rows_per_block;
    const long long r_end = min(r_begin + rows_per_block, BT);
    if (threadIdx.x < kDbiasCols) part[threadIdx.x] = 0.0f;
    float acc[2][8];
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[h][k] = 0.0f;
    const bool in0 = col0 + cv * 8 < OC;
    const bool in1 = col0 + 64 + cv * 8 < OC;
    // four rows per thread in flight (eight 128-bit loads) to cover the DRAM latency
    for (long long r0 = r_begin + warp * 4 + rs; r0 < r_end; r0 += 128) {
        uint4 v0[4], v1[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const long long r = r0 + 32 * i;
            v0[i] = make_uint4(0, 0, 0, 0);
            v1[i] = make_uint4(0, 0, 0, 0);
            if (r < r_end) {
                const __nv_bfloat16 *rowp = dz + r * OC + col0 + cv * 8;
                if (in0) v0[i] = __ldg(reinterpret_cast<const uint4 *>(rowp));
                if (in1) v1[i] = __ldg(reinterpret_cast<const uint4 *>(rowp + 64));
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t a[4] = {v0[i].x, v0[i].y, v0[i].z, v0[i].w};
            const uint32_t b[4] = {v1[i].x, v1[i].y, v1[i].z, v1[i].w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                acc[0][2 * k] += ptx::bf16_lo(a[k]);
                acc[0][2 * k + 1] += ptx::bf16_hi(a[k]);
                acc[1][2 * k] += ptx::bf16_lo(b[k]);
                acc[1][2 * k + 1] += ptx::bf16_hi(b[k]);
            }
        }
    }
    __syncthreads();
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            float v = acc[h][k];
            v += __shfl_xor_sync(0xffffffffu, v, 8);
            v += __shfl_xor_sync(0xffffffffu, v, 16);
            if (rs == 0) atomicAdd(&part[h * 64 + cv * 8 + k], v);
        }
    __syncthreads();
    if (threadIdx.x < kDbiasCols) {
        const int col = col0 + threadIdx.x;
        if (col < OC) atomicAdd(dbias + col, part[threadIdx.x]);
    }
}

// fp32 -> bf16 (round to nearest even), 8 elements per thread per iteration: two 128-bit loads, one
// 128-bit store. HBM-bound: 6 bytes per element.
__global__ void __launch_bounds__(256)
cast_f32_bf16_kernel(__nv_bfloat16 *__restrict__ dst, const float *__restrict__ src, long long n)
{
    const long long nvec = n / 8;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    const long long t0 = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const float4 *s4 = reinterpret_cast<const float4 *>(src);
    uint4 *d4 = reinterpret_cast<uint4 *>(dst);
    for (long long i = t0; i < nvec; i += stride) {
        const float4 a = __ldg(s4 + 2 * i);
        const float4 b = __ldg(s4 + 2 * i + 1);
        d4[i] = make_uint4(ptx::pack_bf16x2(a.x, a.y), ptx::pack_bf16x2(a.z, a.w),
                           ptx::pack_bf16x2(b.x, b.y), ptx::pack_bf16x2(b.z, b.w));
    }
    for (long long i = nvec * 8 + t0; i < n; i += stride) dst[i] = __float2bfloat16_rn(src[i]);
}

// Cross-entropy over the first V columns of the head's logits, from the per-tile softmax statistics
// the forward GEMM wrote: one warp per row combines the partial (max, sum exp) pairs into
// lse = log sum_j exp(logit_j) and loss = lse - logit[target]. A target outside [0, V) gives NaN.
__global__ void __launch_bounds__(256)
ce_reduce_kernel(float *__restrict__ loss, float *__restrict__ lse, const float2 *__restrict__ stats,
                 int stats_ld, const __nv_bfloat16 *__restrict__ logits, long long ld,
                 const int *__restrict__ targets, long long BT, int V)
{
    const int lane = threadIdx.x & 31;
    const long long row = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
    if (row >= BT) return;
    const float2 *st = stats + row * stats_ld;
    float m = -INFINITY;
    for (int k = lane; k < stats_ld; k += 32) m = fmaxf(m, st[k].x);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float s = 0.0f;
    for (int k = lane; k < stats_ld; k += 32) {
        const float2 v = st[k];
        if (v.x > -INFINITY) s += v.y * __expf(v.x - m);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) {
        const float l = m + __logf(s);
        const int t = targets[row];
        lse[row] = l;
        loss[row] = (t >= 0 && t < V) ? l - __bfloat162float(logits[row * ld + t]) : NAN;
    }
}

// dlogits = gscale * (softmax - onehot) on the first V columns, 0 on the padding columns;
// 8 columns per thread (128-bit load and store). May run in place (dlogits == logits).
__global__ void __launch_bounds__(256)
ce_backward_kernel(uint4 *dlogits, const uint4 *logits, const float *__restrict__ lse,
                   const int *__restrict__ targets, float gscale, long long BT, int vec_per_row, int V)
{
    const long long total = BT * vec_per_row;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += stride) {
        const long long row = i / vec_per_row;
        const int col0 = static_cast<int>(i - row * vec_per_row) * 8;
        const uint4 v = logits[i];
        const float l = lse[row] * 1.4426950408889634f;
        const int t = targets[row];
        const uint32_t x[4] = {v.x, v.y, v.z, v.w};
        uint32_t o[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int c = col0 + 2 * k;
            float p0 = ptx::ex2_approx(fmaf(ptx::bf16_lo(x[k]), 1.4426950408889634f, -l));
            float p1 = ptx::ex2_approx(fmaf(ptx::bf16_hi(x[k]), 1.4426950408889634f, -l));
            p0 = (c < V) ? gscale * (p0 - (c == t ? 1.0f : 0.0f)) : 0.0f;
            p1 = (c + 1 < V) ? gscale * (p1 - (c + 1 == t ? 1.0f : 0.0f)) : 0.0f;
            o[k] = ptx::pack_bf16x2(p0, p1);
        }
        dlogits[i] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// Waits on a barrier that nothing signals, for at most limit_ns, then leaves normally.
__global__ void wait_timeout_kernel(int *status, unsigned long long limit_ns)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&bar), 1);
        abort_flag = 0;
        ptx::fence_barrier_init();
        const WaitCtx w{ptx::smem_u32(&abort_flag), status, limit_ns};
        (void)wait_barrier(w, ptx::smem_u32(&bar), 0, 900);
    }
}

}  // namespace nb
