// CUDA-core (FFMA) linear + epilogue (+ row-norm) kernels: the fp32 path, and the generic path for
// bf16 calls whose pointers or sizes rule out TMA.  fp32 stays off the tensor cores on purpose:
// single-pass TF32 keeps 10 mantissa bits and misses the 1e-4 absolute gate of the fp32 calls.
//
// row-resident kernel: a CTA of 256 threads owns BM whole rows (N <= 2048), thread t holds the
//   accumulators of columns t, t+256, ...; W streams through shared memory in [256 x 32] slabs;
//   the row statistics are reduced inside the CTA and the row is normalised before its only store.
// tiled kernel: classic 64x64x16 register-tiled GEMM (4x4 per thread) with the element-wise
//   epilogue; a row-norm, if any, follows as a separate in-place row kernel.
#include "kf_common.cuh"

namespace kf {
namespace {

constexpr int kThreads = 256;
constexpr int kSlabK = 32;

template <typename T>
__device__ __forceinline__ float epilogue_elem(float acc, long long m, long long n, const T* bias, const T* res,
                                               long long ldr, int act, float scale) {
    float z = acc;
    if (bias) z += Elem<T>::load(bias + n);
    float a = apply_act<true>(act, z) * scale;
    if (res) a += Elem<T>::load(res + m * ldr + n);
    return a;
}

// ------------------------------------------------------------------------------ row-resident
template <typename T, int BM, int NPT>
__global__ void __launch_bounds__(kThreads)
simt_rows_kernel(const T* __restrict__ X, long long ldx, const T* __restrict__ W, long long ldw, T* Y,
                 long long ldy, int M, int N, int K, const T* __restrict__ bias, const T* res, long long ldr,
                 int act, float scale, int norm, const T* __restrict__ gamma, const T* __restrict__ beta,
                 float eps) {
    __shared__ float ws[kThreads][kSlabK + 1];
    __shared__ float xs[BM][kSlabK];
    __shared__ float red[kThreads / 32][BM];
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int m0 = blockIdx.x * BM;

    float acc[BM][NPT];
#pragma unroll
    for (int i = 0; i < BM; ++i)
#pragma unroll
        for (int j = 0; j < NPT; ++j) acc[i][j] = 0.f;

    // Software pipeline over (k0, j) steps: the global loads of the next step are issued before the
    // FMAs of the current one, so their latency hides behind the arithmetic and the barriers.
    static_assert(BM * kSlabK <= kThreads, "one X element per thread and step");
    auto load_w = [&](float (&tmp)[32], int k0, int j) {
#pragma unroll
        for (int u = 0; u < 32; ++u) {
            const int n = j * kThreads + u * (kThreads / 32) + warp;      // a warp reads one W row per step (coalesced)
            tmp[u] = (n < N && k0 + lane < K) ? Elem<T>::load(W + (long long)n * ldw + k0 + lane) : 0.f;
        }
    };
    auto load_x = [&](int k0) -> float {
        const int i = t / kSlabK, kk = t % kSlabK;
        return (t < BM * kSlabK && m0 + i < M && k0 + kk < K) ? Elem<T>::load(X + (long long)(m0 + i) * ldx + k0 + kk) : 0.f;
    };
    float tmp[32];
    float xv = 0.f;
    if (K > 0) {
        load_w(tmp, 0, 0);
        xv = load_x(0);
    }
    for (int k0 = 0; k0 < K; k0 += kSlabK) {
#pragma unroll
        for (int j = 0; j < NPT; ++j) {
            __syncthreads();                               // the previous step's FMAs are done with ws / xs
#pragma unroll
            for (int u = 0; u < 32; ++u) ws[u * (kThreads / 32) + warp][lane] = tmp[u];
            if (j == 0 && t < BM * kSlabK) xs[t / kSlabK][t % kSlabK] = xv;
            __syncthreads();
            if (j + 1 < NPT) {
                load_w(tmp, k0, j + 1);
            } else if (k0 + kSlabK < K) {
                load_w(tmp, k0 + kSlabK, 0);
                xv = load_x(k0 + kSlabK);
            }
#pragma unroll
            for (int kk = 0; kk < kSlabK; ++kk) {
                const float w = ws[t][kk];
#pragma unroll
                for (int i = 0; i < BM; ++i) acc[i][j] = fmaf(xs[i][kk], w, acc[i][j]);
            }
        }
    }

    // element-wise epilogue, in place in the accumulators
#pragma unroll
    for (int i = 0; i < BM; ++i)
#pragma unroll
        for (int j = 0; j < NPT; ++j) {
            const int n = j * kThreads + t;
            if (m0 + i < M && n < N) acc[i][j] = epilogue_elem<T>(acc[i][j], m0 + i, n, bias, res, ldr, act, scale);
        }

    auto block_reduce = [&](float (&v)[BM], bool is_max) {
#pragma unroll
        for (int i = 0; i < BM; ++i) v[i] = is_max ? warp_max(v[i]) : warp_sum(v[i]);
        __syncthreads();
        if (lane == 0)
#pragma unroll
            for (int i = 0; i < BM; ++i) red[warp][i] = v[i];
        __syncthreads();
#pragma unroll
        for (int i = 0; i < BM; ++i) {
            float r = red[0][i];
            for (int w = 1; w < kThreads / 32; ++w) r = is_max ? fmaxf(r, red[w][i]) : r + red[w][i];
            v[i] = r;
        }
    };

    float s0[BM], s1[BM];
    if (norm == KF_NORM_SOFTMAX) {
#pragma unroll
        for (int i = 0; i < BM; ++i) {
            s0[i] = -INFINITY;
#pragma unroll
            for (int j = 0; j < NPT; ++j)
                if (j * kThreads + t < N) s0[i] = fmaxf(s0[i], acc[i][j]);
        }
        block_reduce(s0, true);
#pragma unroll
        for (int i = 0; i < BM; ++i) {
            s1[i] = 0.f;
#pragma unroll
            for (int j = 0; j < NPT; ++j)
                if (j * kThreads + t < N) {
                    acc[i][j] = expf(acc[i][j] - s0[i]);
                    s1[i] += acc[i][j];
                }
        }
        block_reduce(s1, false);
#pragma unroll
        for (int i = 0; i < BM; ++i) {
            const float inv = 1.0f / s1[i];
#pragma unroll
            for (int j = 0; j < NPT; ++j) acc[i][j] *= inv;
        }
    } else if (norm == KF_NORM_LAYERNORM || norm == KF_NORM_RMSNORM) {
#pragma unroll
        for (int i = 0; i < BM; ++i) {
            s0[i] = 0.f;
            if (norm == KF_NORM_LAYERNORM) {
#pragma unroll
                for (int j = 0; j < NPT; ++j)
                    if (j * kThreads + t < N) s0[i] += acc[i][j];
            }
        }
        if (norm == KF_NORM_LAYERNORM) {
            block_reduce(s0, false);
#pragma unroll
            for (int i = 0; i < BM; ++i) s0[i] /= (float)N;
        }
#pragma unroll
        for (int i = 0; i < BM; ++i) {
            s1[i] = 0.f;
#pragma unroll
            for (int j = 0; j < NPT; ++j)
                if (j * kThreads + t < N) {
                    const float d = acc[i][j] - s0[i];
                    s1[i] = fmaf(d, d, s1[i]);
                }
        }
        block_reduce(s1, false);
#pragma unroll
        for (int j = 0; j < NPT; ++j) {
            const int n = j * kThreads + t;
            if (n < N) {
                const float g = gamma ? Elem<T>::load(gamma + n) : 1.0f;
                const float b = (beta && norm == KF_NORM_LAYERNORM) ? Elem<T>::load(beta + n) : 0.0f;
#pragma unroll
                for (int i = 0; i < BM; ++i) {
                    const float rstd = 1.0f / sqrtf(s1[i] / (float)N + eps);
                    acc[i][j] = (acc[i][j] - s0[i]) * rstd * g + b;
                }
            }
        }
    }
#pragma unroll
    for (int i = 0; i < BM; ++i)
#pragma unroll
        for (int j = 0; j < NPT; ++j) {
            const int n = j * kThreads + t;
            if (m0 + i < M && n < N) Elem<T>::store(Y + (long long)(m0 + i) * ldy + n, acc[i][j]);
        }
}

// ------------------------------------------------------------------------------ tiled 64x64x16
constexpr int kTM = 64, kTN = 64, kTK = 16, kPad = 4;

template <typename T>
__global__ void __launch_bounds__(kThreads)
simt_tiled_kernel(const T* __restrict__ X, long long ldx, const T* __restrict__ W, long long ldw, T* Y,
                  long long ldy, long long M, long long N, long long K, const T* __restrict__ bias, const T* res,
                  long long ldr, int act, float scale) {
    __shared__ float As[kTK][kTM + kPad];
    __shared__ float Bs[kTK][kTN + kPad];
    const int t = threadIdx.x;
    const int tx = t % 16, ty = t / 16;                 // 16 x 16 threads, 4 x 4 outputs each
    const long long m0 = (long long)blockIdx.y * kTM, n0 = (long long)blockIdx.x * kTN;
    const int lrow = t / 4, lk = (t % 4) * 4;           // loader: 64 rows x 16 k, 4 k per thread

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (long long k0 = 0; k0 < K; k0 += kTK) {
        __syncthreads();
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const long long k = k0 + lk + q;
            As[lk + q][lrow] = (m0 + lrow < M && k < K) ? Elem<T>::load(X + (m0 + lrow) * ldx + k) : 0.f;
            Bs[lk + q][lrow] = (n0 + lrow < N && k < K) ? Elem<T>::load(W + (n0 + lrow) * ldw + k) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kTK; ++kk) {
            const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
            const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const long long m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const long long n = n0 + tx * 4 + j;
            if (n < N) Elem<T>::store(Y + m * ldy + n, epilogue_elem<T>(acc[i][j], m, n, bias, res, ldr, act, scale));
        }
    }
}

// ------------------------------------------------------------------------------ tiled 128x128x16
// The same contract as the 64x64 kernel for problems with enough 128 x 128 tiles to fill the device: 8 x 8
// outputs per thread (two groups of 4 rows and of 4 columns, 64 apart, so that the 16-byte shared-memory
// reads of a quarter-warp are contiguous), and the next k-slab on its way from global memory into
// registers while the current one is multiplied out of shared memory.
constexpr int kBM2 = 128, kBN2 = 128, kBK2 = 16;

template <typename T>
__global__ void __launch_bounds__(kThreads, 2)
simt_tiled128_kernel(const T* __restrict__ X, long long ldx, const T* __restrict__ W, long long ldw, T* Y,
                     long long ldy, long long M, long long N, long long K, const T* __restrict__ bias, const T* res,
                     long long ldr, int act, float scale) {
    __shared__ __align__(16) float As[2][kBK2][kBM2];
    __shared__ __align__(16) float Bs[2][kBK2][kBN2];
    const int t = threadIdx.x;
    const int tx = t % 16, ty = t / 16;
    const long long m0 = (long long)blockIdx.y * kBM2, n0 = (long long)blockIdx.x * kBN2;
    const int lrow = t / 2, lk = (t % 2) * 8;           // loader: 128 rows x 16 k, 8 consecutive k per thread
    const bool a_ok = m0 + lrow < M, b_ok = n0 + lrow < N;
    const T* xa = X + (m0 + lrow) * ldx;
    const T* wb = W + (n0 + lrow) * ldw;

    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

    float ra[8], rb[8];
    auto fetch = [&](long long k0) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const long long k = k0 + lk + q;
            ra[q] = (a_ok && k < K) ? Elem<T>::load(xa + k) : 0.f;
            rb[q] = (b_ok && k < K) ? Elem<T>::load(wb + k) : 0.f;
        }
    };
    auto stash = [&](int buf) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            As[buf][lk + q][lrow] = ra[q];
            Bs[buf][lk + q][lrow] = rb[q];
        }
    };
    if (K > 0) {
        fetch(0);
        stash(0);
    }
    __syncthreads();
    int buf = 0;
    for (long long k0 = 0; k0 < K; k0 += kBK2, buf ^= 1) {
        const bool more = k0 + kBK2 < K;
        if (more) fetch(k0 + kBK2);                      // in flight during the arithmetic below
#pragma unroll
        for (int kk = 0; kk < kBK2; ++kk) {
            const float4 a0 = *reinterpret_cast<const float4*>(&As[buf][kk][ty * 4]);
            const float4 a1 = *reinterpret_cast<const float4*>(&As[buf][kk][64 + ty * 4]);
            const float4 b0 = *reinterpret_cast<const float4*>(&Bs[buf][kk][tx * 4]);
            const float4 b1 = *reinterpret_cast<const float4*>(&Bs[buf][kk][64 + tx * 4]);
            const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        if (more) stash(buf ^ 1);                        // the other buffer was last read before the previous barrier
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const long long m = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const long long n = n0 + (j < 4 ? tx * 4 + j : 64 + tx * 4 + (j - 4));
            if (n < N) Elem<T>::store(Y + m * ldy + n, epilogue_elem<T>(acc[i][j], m, n, bias, res, ldr, act, scale));
        }
    }
}

template <typename T, int BM, int NPT>
cudaError_t launch_rows(const T* X, long long ldx, const T* W, long long ldw, T* Y, long long ldy, long long M,
                        long long N, long long K, const EpilogueParams& ep, const RowNormParams& rn,
                        cudaStream_t st, int* grid_out) {
    const long long ctas = (M + BM - 1) / BM;
    if (ctas > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    if (grid_out) *grid_out = (int)ctas;
    simt_rows_kernel<T, BM, NPT><<<(unsigned)ctas, kThreads, 0, st>>>(
        X, ldx, W, ldw, Y, ldy, (int)M, (int)N, (int)K, static_cast<const T*>(ep.bias),
        static_cast<const T*>(ep.residual), ep.ldr, ep.act, ep.scale, rn.norm, static_cast<const T*>(rn.gamma),
        static_cast<const T*>(rn.beta), rn.eps);
    return cudaGetLastError();
}

template <typename T, int NPT>
cudaError_t launch_rows_bm(const T* X, long long ldx, const T* W, long long ldw, T* Y, long long ldy,
                           long long M, long long N, long long K, const EpilogueParams& ep,
                           const RowNormParams& rn, cudaStream_t st, int* grid_out) {
    // rows per CTA: fewest rows that still keep the grid within about two waves of 148 SMs
    int bm = 1;
    while (bm < 8 && bm * NPT < 16 && (M + bm - 1) / bm > 2 * 148) bm <<= 1;
    switch (bm) {
    case 1: return launch_rows<T, 1, NPT>(X, ldx, W, ldw, Y, ldy, M, N, K, ep, rn, st, grid_out);
    case 2: return launch_rows<T, 2, NPT>(X, ldx, W, ldw, Y, ldy, M, N, K, ep, rn, st, grid_out);
    case 4: return launch_rows<T, 4, NPT>(X, ldx, W, ldw, Y, ldy, M, N, K, ep, rn, st, grid_out);
    default: return launch_rows<T, 8, NPT>(X, ldx, W, ldw, Y, ldy, M, N, K, ep, rn, st, grid_out);
    }
}

template <typename T>
cudaError_t launch_typed(const void* Xv, long long ldx, const void* Wv, long long ldw, void* Yv, long long ldy,
                         long long M, long long N, long long K, const EpilogueParams& ep, const RowNormParams& rn,
                         bool row_resident, cudaStream_t st, int* grid_out) {
    const T* X = static_cast<const T*>(Xv);
    const T* W = static_cast<const T*>(Wv);
    T* Y = static_cast<T*>(Yv);
    if (row_resident) {
        if (N <= 256) return launch_rows_bm<T, 1>(X, ldx, W, ldw, Y, ldy, M, N, K, ep, rn, st, grid_out);
        if (N <= 512) return launch_rows_bm<T, 2>(X, ldx, W, ldw, Y, ldy, M, N, K, ep, rn, st, grid_out);
        if (N <= 1024) return launch_rows_bm<T, 4>(X, ldx, W, ldw, Y, ldy, M, N, K, ep, rn, st, grid_out);
        return launch_rows_bm<T, 8>(X, ldx, W, ldw, Y, ldy, M, N, K, ep, rn, st, grid_out);
    }
    // 128 x 128 tiles once there are a few dozen of them (8 x 8 outputs per thread: a quarter of the
    // shared-memory traffic per multiply-add, and the next slab prefetched), else 64 x 64
    const long long gx2 = (N + kBN2 - 1) / kBN2, gy2 = (M + kBM2 - 1) / kBM2;
    if (gx2 * gy2 >= 24 && gy2 <= 65535 && gx2 <= 0x7FFFFFFFll) {
        if (grid_out) *grid_out = (int)(gx2 * gy2);
        simt_tiled128_kernel<T><<<dim3((unsigned)gx2, (unsigned)gy2), kThreads, 0, st>>>(
            X, ldx, W, ldw, Y, ldy, M, N, K, static_cast<const T*>(ep.bias), static_cast<const T*>(ep.residual),
            ep.ldr, ep.act, ep.scale);
    } else {
        const long long gx = (N + kTN - 1) / kTN, gy = (M + kTM - 1) / kTM;
        if (gx > 0x7FFFFFFFll || gy > 65535) return cudaErrorInvalidConfiguration;
        if (grid_out) *grid_out = (int)(gx * gy);
        simt_tiled_kernel<T><<<dim3((unsigned)gx, (unsigned)gy), kThreads, 0, st>>>(
            X, ldx, W, ldw, Y, ldy, M, N, K, static_cast<const T*>(ep.bias), static_cast<const T*>(ep.residual),
            ep.ldr, ep.act, ep.scale);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || rn.norm == KF_NORM_NONE) return e;
    return launch_row_norm(Yv, ldy, Yv, ldy, M, N, sizeof(T) == 4 ? KF_F32 : KF_BF16, rn, st);
}

}  // namespace

bool simt_row_resident_ok(long long N) { return N <= 8 * kThreads; }

cudaError_t launch_simt_linear(const void* X, long long ldx, const void* W, long long ldw, void* Y,
                               long long ldy, long long M, long long N, long long K, int dt,
                               const EpilogueParams& ep, const RowNormParams& rn, bool row_resident,
                               cudaStream_t st, int* grid_out) {
    if (dt == KF_F32)
        return launch_typed<float>(X, ldx, W, ldw, Y, ldy, M, N, K, ep, rn, row_resident, st, grid_out);
    return launch_typed<__nv_bfloat16>(X, ldx, W, ldw, Y, ldy, M, N, K, ep, rn, row_resident, st, grid_out);
}

}  // namespace kf
