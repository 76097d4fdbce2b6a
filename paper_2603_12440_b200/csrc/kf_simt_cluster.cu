// Small fp32 linear + epilogue + row-norm calls (M <= 512, N <= 512, below the tensor-core gate): latency decides
// them, not throughput, so the work of a row is spread over a thread-block cluster instead of held in one CTA.
//
//   cluster of 8 CTAs = 8 rows x all N columns; CTA r owns columns [r NC, (r+1) NC), NC = ceil(N / 8)
//   CTA of 8 warps: a slab of its W slice (NC columns x 256 / CPL k) and of the 8 X rows goes to shared memory
//   through registers, every load of a slab in flight at once (for K <= 256 that is the whole problem in
//   one round trip); warp w then multiplies the w-th eighth of the slab's k range for all 8 rows, lane =
//   column, so each W value leaves shared memory once; the eight partial sums of an output are added in
//   a fixed order through shared memory, after which warp = row, lane = column.
//   row statistics: each CTA reduces its slice of the 8 rows (one warp per row) to one float2 per row in its
//   own shared memory -- softmax (max, sum of exp about it), LayerNorm (mean, sum of squared deviations;
//   Chan's merge), RMSNorm (sum of squares) -- and after one cluster barrier reads the other seven CTAs'
//   pairs through distributed shared memory; a second barrier, whose wait is the last thing a CTA does,
//   keeps every CTA's shared memory alive until all have read it.
#include <cooperative_groups.h>

#include "kf_common.cuh"

namespace cg = cooperative_groups;

namespace kf {
namespace {

constexpr int kCl = 8;               // CTAs per cluster
constexpr int kRowsCl = 8;           // rows per cluster, one warp each after the K loop
constexpr int kThreadsCl = 256;

template <int CPL>                   // columns per lane: 1 (NC <= 32) or 2 (NC <= 64)
__global__ void __launch_bounds__(kThreadsCl, 2)     // two CTAs per SM: a GPC then holds two clusters per 8 SMs
simt_cluster_kernel(const float* __restrict__ X, long long ldx, const float* __restrict__ W, long long ldw, float* Y,
                    long long ldy, int M, int N, int K, const float* __restrict__ bias, const float* res,
                    long long ldr, int act, float scale, int norm, const float* __restrict__ gamma,
                    const float* __restrict__ beta, float eps) {
    constexpr int KS = 256 / CPL;            // k per slab
    constexpr int NCOLS = 32 * CPL;          // columns of a CTA's slice (upper bound)
    constexpr int KQ = KS / 4;               // float4 per slab row
    constexpr int PQ = KQ + 1;               // row pitch of the W slab in float4: lanes 0..7 of a 16-byte read hit 32 banks
    constexpr int WU = NCOLS * KQ / kThreadsCl;      // float4 of W per thread and slab (8)
    constexpr int XU = kRowsCl * KQ / kThreadsCl;    // float4 of X per thread and slab (2 or 1)
    constexpr int KW = KQ / 8;               // float4 steps of one warp per slab
    static_assert(NCOLS * PQ >= 8 * kRowsCl * NCOLS / 4, "the partial sums reuse the W slab");
    __shared__ float4 ws4[NCOLS * PQ];
    __shared__ float4 xs4[kRowsCl * KQ];
    __shared__ float2 exch[kRowsCl];

    cg::cluster_group cluster = cg::this_cluster();
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int rank = (int)(blockIdx.x % kCl);                // = the CTA's rank in its cluster (1-D clusters of kCl)
    const int m0 = (int)(blockIdx.x / kCl) * kRowsCl;
    const int NC = (N + kCl - 1) / kCl;
    const int n_base = rank * NC;
    const int ncols = max(0, min(NC, N - n_base));           // columns this CTA really has
    float4 wreg[WU], xreg[XU];
    auto load_slab = [&](int k0) {
#pragma unroll
        for (int u = 0; u < WU; ++u) {
            const int f = t + u * kThreadsCl, col = f / KQ, k = k0 + 4 * (f % KQ);
            wreg[u] = (col < ncols && k < K) ? __ldg(reinterpret_cast<const float4*>(W + (long long)(n_base + col) * ldw + k))
                                             : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < XU; ++u) {
            const int f = t + u * kThreadsCl, r = f / KQ, k = k0 + 4 * (f % KQ);
            xreg[u] = (m0 + r < M && k < K) ? __ldg(reinterpret_cast<const float4*>(X + (long long)(m0 + r) * ldx + k))
                                            : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };

    float acc[kRowsCl][CPL];
#pragma unroll
    for (int r = 0; r < kRowsCl; ++r)
#pragma unroll
        for (int j = 0; j < CPL; ++j) acc[r][j] = 0.f;

    if (K > 0) load_slab(0);
    for (int k0 = 0; k0 < K; k0 += KS) {
        __syncthreads();                                     // the previous slab has been consumed
#pragma unroll
        for (int u = 0; u < WU; ++u) {
            const int f = t + u * kThreadsCl;
            ws4[(f / KQ) * PQ + f % KQ] = wreg[u];
        }
#pragma unroll
        for (int u = 0; u < XU; ++u) xs4[t + u * kThreadsCl] = xreg[u];
        __syncthreads();
        if (k0 + KS < K) load_slab(k0 + KS);                 // in flight during the arithmetic below
#pragma unroll
        for (int i = 0; i < KW; ++i) {
            const int kq = warp * KW + i;
            float4 w[CPL];
#pragma unroll
            for (int j = 0; j < CPL; ++j) w[j] = ws4[(lane + 32 * j) * PQ + kq];
#pragma unroll
            for (int r = 0; r < kRowsCl; ++r) {
                const float4 x = xs4[r * KQ + kq];           // same address in every lane: a broadcast
#pragma unroll
                for (int j = 0; j < CPL; ++j) {
                    acc[r][j] = fmaf(x.x, w[j].x, acc[r][j]);
                    acc[r][j] = fmaf(x.y, w[j].y, acc[r][j]);
                    acc[r][j] = fmaf(x.z, w[j].z, acc[r][j]);
                    acc[r][j] = fmaf(x.w, w[j].w, acc[r][j]);
                }
            }
        }
    }

    // the eight k-range partials of every output, added in warp order; from here on warp = row, lane = column
    __syncthreads();
    float* red = reinterpret_cast<float*>(ws4);              // [k-range warp][row][column]
#pragma unroll
    for (int r = 0; r < kRowsCl; ++r)
#pragma unroll
        for (int j = 0; j < CPL; ++j) red[(warp * kRowsCl + r) * NCOLS + lane + 32 * j] = acc[r][j];
    __syncthreads();
    const int row = m0 + warp;
    float a[CPL];
    bool ok[CPL];
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
        const int c = lane + 32 * j;
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) s += red[(w * kRowsCl + warp) * NCOLS + c];
        ok[j] = row < M && c < ncols;
        a[j] = 0.f;
        if (ok[j]) {
            const int n = n_base + c;
            float z = s;
            if (bias) z += __ldg(bias + n);
            a[j] = apply_act<true>(act, z) * scale;
            if (res) a[j] += res[(long long)row * ldr + n];
        }
    }

    if (norm != KF_NORM_NONE) {
        // this CTA's share of the row statistics
        float2 mine = make_float2(0.f, 0.f);
        float e[CPL];
        if (norm == KF_NORM_SOFTMAX) {
            float m = -INFINITY;
#pragma unroll
            for (int j = 0; j < CPL; ++j)
                if (ok[j]) m = fmaxf(m, a[j]);
            m = warp_max(m);
            float s = 0.f;
#pragma unroll
            for (int j = 0; j < CPL; ++j) {
                e[j] = ok[j] ? expf(a[j] - m) : 0.f;
                s += e[j];
            }
            mine = make_float2(m, warp_sum(s));
        } else if (norm == KF_NORM_LAYERNORM) {
            float s = 0.f;
#pragma unroll
            for (int j = 0; j < CPL; ++j) s += ok[j] ? a[j] : 0.f;
            const float mu = ncols > 0 ? warp_sum(s) / (float)ncols : 0.f;
            float q = 0.f;
#pragma unroll
            for (int j = 0; j < CPL; ++j) {
                const float d = ok[j] ? a[j] - mu : 0.f;
                q = fmaf(d, d, q);
            }
            mine = make_float2(mu, warp_sum(q));
        } else {
            float q = 0.f;
#pragma unroll
            for (int j = 0; j < CPL; ++j) q = fmaf(a[j], a[j], q);           // a is 0 where there is no column
            mine = make_float2(0.f, warp_sum(q));
        }
        // every CTA publishes its pairs in its own shared memory; after the barrier (which also says that every
        // CTA of the cluster is running) lane p reads CTA p's pair of this row, and the warp shares them out
        if (lane == 0) exch[warp] = mine;
        cluster.sync();
        const float2 theirs = lane < kCl ? *cluster.map_shared_rank(&exch[warp], lane) : make_float2(0.f, 0.f);
        cluster.barrier_arrive();                            // this CTA has read; waited for before it exits
        float2 part[kCl];
#pragma unroll
        for (int p = 0; p < kCl; ++p)
            part[p] = make_float2(__shfl_sync(0xFFFFFFFFu, theirs.x, p), __shfl_sync(0xFFFFFFFFu, theirs.y, p));
        if (norm == KF_NORM_SOFTMAX) {
            float m = part[0].x;                             // CTA 0 always has a column
#pragma unroll
            for (int p = 1; p < kCl; ++p) m = fmaxf(m, part[p].x);
            float l = 0.f;
#pragma unroll
            for (int p = 0; p < kCl; ++p)
                if (part[p].y > 0.f) l = fmaf(part[p].y, expf(part[p].x - m), l);
            const float f = expf(mine.x - m) / l;
#pragma unroll
            for (int j = 0; j < CPL; ++j) a[j] = e[j] * f;
        } else {
            float mu = 0.f, q = 0.f;
            if (norm == KF_NORM_LAYERNORM) {
#pragma unroll
                for (int p = 0; p < kCl; ++p) mu = fmaf((float)max(0, min(NC, N - p * NC)), part[p].x, mu);
                mu /= (float)N;
            }
#pragma unroll
            for (int p = 0; p < kCl; ++p) {
                const float cnt = (float)max(0, min(NC, N - p * NC)), d = part[p].x - mu;
                q += part[p].y + (norm == KF_NORM_LAYERNORM ? cnt * d * d : 0.f);
            }
            const float rstd = 1.0f / sqrtf(q / (float)N + eps);
#pragma unroll
            for (int j = 0; j < CPL; ++j)
                if (ok[j]) {
                    const int n = n_base + lane + 32 * j;
                    const float g = gamma ? __ldg(gamma + n) : 1.0f;
                    const float b = (beta && norm == KF_NORM_LAYERNORM) ? __ldg(beta + n) : 0.0f;
                    a[j] = (a[j] - mu) * rstd * g + b;
                }
        }
    }
#pragma unroll
    for (int j = 0; j < CPL; ++j)
        if (ok[j]) Y[(long long)row * ldy + n_base + lane + 32 * j] = a[j];
    if (norm != KF_NORM_NONE) cluster.barrier_wait();        // no CTA leaves while another may still read its pairs
}

template <int CPL>
cudaError_t launch_cluster(const float* X, long long ldx, const float* W, long long ldw, float* Y, long long ldy,
                           long long M, long long N, long long K, const EpilogueParams& ep, const RowNormParams& rn,
                           cudaStream_t st, int* grid_out) {
    const long long ctas = ((M + kRowsCl - 1) / kRowsCl) * kCl;
    if (ctas > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    if (grid_out) *grid_out = (int)ctas;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)ctas);
    lc.blockDim = dim3(kThreadsCl);
    lc.dynamicSmemBytes = 0;
    lc.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = kCl;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    lc.attrs = at;
    lc.numAttrs = rn.norm != KF_NORM_NONE ? 1 : 0;           // without a row-norm nothing crosses CTAs: a plain grid
    return cudaLaunchKernelEx(&lc, simt_cluster_kernel<CPL>, X, ldx, W, ldw, Y, ldy, (int)M, (int)N, (int)K,
                              static_cast<const float*>(ep.bias), static_cast<const float*>(ep.residual), ep.ldr,
                              ep.act, ep.scale, rn.norm, static_cast<const float*>(rn.gamma),
                              static_cast<const float*>(rn.beta), rn.eps);
}

}  // namespace

// fp32 with 16-byte aligned rows (the caller checks pointers and pitches) and K a multiple of 4; rows of 64 to
// 512 columns (shorter ones would leave most lanes of a CTA without a column).  Only where latency decides:
// at most 512 rows (64 clusters) -- a cluster of 8 needs 8 SMs of one GPC at the same time, so a B200 holds
// two clusters per GPC and CTA slot (the kernel is kept to 128 registers for two CTAs per SM: with one, C1's
// 16 clusters ran in two waves, 14.3 us instead of 10.2), and further clusters wait for whole clusters to
// leave (1024 x 256 x 112 with softmax: 29 us here, 16 for the row-resident kernel; 512 x 512 x 112: 16 here,
// 22 there; 64 x 512 x 900: 20 here, 104 there) -- and a W of at least 64 KiB, below which the row-resident
// kernel's single CTA per row reads it as quickly (16 x 64 x 16: 8 us either way)
bool simt_cluster_ok(long long M, long long N, long long K) {
    return N >= 64 && N <= kCl * 64 && K % 4 == 0 && M <= 512 && N * K >= 16384;
}

cudaError_t launch_simt_cluster(const void* X, long long ldx, const void* W, long long ldw, void* Y, long long ldy,
                                long long M, long long N, long long K, const EpilogueParams& ep,
                                const RowNormParams& rn, cudaStream_t st, int* grid_out) {
    const float* x = static_cast<const float*>(X);
    const float* w = static_cast<const float*>(W);
    float* y = static_cast<float*>(Y);
    if ((N + kCl - 1) / kCl <= 32) return launch_cluster<1>(x, ldx, w, ldw, y, ldy, M, N, K, ep, rn, st, grid_out);
    return launch_cluster<2>(x, ldx, w, ldw, y, ldy, M, N, K, ep, rn, st, grid_out);
}

}  // namespace kf
