// Stand-alone row operators (softmax, LayerNorm, RMSNorm) on an existing [M,N]: memory-bound.
//
// Fast path: a row lives in the registers of TPR threads as VPT 16-byte vectors each, so every
// element is read from HBM once and written once (streaming loads/stores, 128-bit, coalesced);
// statistics use warp shuffles, plus one shared-memory hop when a row spans several warps.
// LayerNorm takes the mean first and the centred sum of squares second, both from registers.
// Generic path (row length or pointers not 16-byte friendly, or rows too long for registers):
// one CTA per row, scalar accesses, three passes over global memory.
#include "kf_common.cuh"

#include <cstdlib>

namespace kf {
namespace {

constexpr int kRowThreads = 256;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) { __stcs(p, v); }

// reduce over the TPR threads that share a row; `red` has one float per warp of the CTA
template <bool IS_MAX>
__device__ __forceinline__ float group_reduce(float v, int tpr, float* red) {
    v = IS_MAX ? warp_max(v) : warp_sum(v);
    if (tpr <= 32) return v;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wpg = tpr >> 5, g0 = (warp / wpg) * wpg;
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float t = red[g0];
    for (int i = 1; i < wpg; ++i) t = IS_MAX ? fmaxf(t, red[g0 + i]) : t + red[g0 + i];
    return t;
}

template <typename T, int NORM, int VPT>
__global__ void __launch_bounds__(512)
row_norm_reg_kernel(const T* X, long long ldx, T* Y, long long ldy, long long M,   // Y may alias X
                    int N, int tpr, const T* __restrict__ gamma, const T* __restrict__ beta, float eps) {
    constexpr int E = Elem<T>::kVec;
    __shared__ float red[32];
    const int rows_per_cta = blockDim.x / tpr;
    const long long row = (long long)blockIdx.x * rows_per_cta + threadIdx.x / tpr;
    const int lr = threadIdx.x % tpr;
    const int NV = N / E;
    const bool live = row < M;
    const uint4* xr = reinterpret_cast<const uint4*>(X + (live ? row : 0) * ldx);
    uint4* yr = reinterpret_cast<uint4*>(Y + (live ? row : 0) * ldy);

    uint4 v[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int idx = lr + i * tpr;
        v[i] = (live && idx < NV) ? ld_stream(xr + idx) : make_uint4(0, 0, 0, 0);
    }
    float f[E];
    if (NORM == KF_NORM_SOFTMAX) {
        float m = -INFINITY;
#pragma unroll
        for (int i = 0; i < VPT; ++i)
            if (lr + i * tpr < NV) {
                unpack<T>(v[i], f);
#pragma unroll
                for (int e = 0; e < E; ++e) m = fmaxf(m, f[e]);
            }
        m = group_reduce<true>(m, tpr, red);
        const float ms = m * kLog2e;
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < VPT; ++i)
            if (lr + i * tpr < NV) {
                unpack<T>(v[i], f);
#pragma unroll
                for (int e = 0; e < E; ++e) s += exp2f(fmaf(f[e], kLog2e, -ms));
            }
        s = group_reduce<false>(s, tpr, red);
        const float inv = 1.0f / s;
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int idx = lr + i * tpr;
            if (live && idx < NV) {
                unpack<T>(v[i], f);
#pragma unroll
                for (int e = 0; e < E; ++e) f[e] = exp2f(fmaf(f[e], kLog2e, -ms)) * inv;
                st_stream(yr + idx, pack<T>(f));
            }
        }
    } else {
        float mean = 0.f;
        if (NORM == KF_NORM_LAYERNORM) {
            float s = 0.f;
#pragma unroll
            for (int i = 0; i < VPT; ++i)
                if (lr + i * tpr < NV) {
                    unpack<T>(v[i], f);
#pragma unroll
                    for (int e = 0; e < E; ++e) s += f[e];
                }
            mean = group_reduce<false>(s, tpr, red) / (float)N;
        }
        float q = 0.f;
#pragma unroll
        for (int i = 0; i < VPT; ++i)
            if (lr + i * tpr < NV) {
                unpack<T>(v[i], f);
#pragma unroll
                for (int e = 0; e < E; ++e) { const float d = f[e] - mean; q = fmaf(d, d, q); }
            }
        q = group_reduce<false>(q, tpr, red);
        const float rstd = rsqrtf(q / (float)N + eps);
        const uint4* gv = reinterpret_cast<const uint4*>(gamma);
        const uint4* bv = reinterpret_cast<const uint4*>(beta);
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int idx = lr + i * tpr;
            if (live && idx < NV) {
                unpack<T>(v[i], f);
                float g[E], b[E];
                if (gamma) unpack<T>(__ldg(gv + idx), g);
                if (beta && NORM == KF_NORM_LAYERNORM) unpack<T>(__ldg(bv + idx), b);
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    float o = (f[e] - mean) * rstd;
                    if (gamma) o *= g[e];
                    if (beta && NORM == KF_NORM_LAYERNORM) o += b[e];
                    f[e] = o;
                }
                st_stream(yr + idx, pack<T>(f));
            }
        }
    }
}

// generic: one CTA per row, scalar accesses, any N / alignment; Y may alias X
template <typename T, int NORM>
__global__ void __launch_bounds__(kRowThreads)
row_norm_generic_kernel(const T* X, long long ldx, T* Y, long long ldy, long long N,
                        const T* __restrict__ gamma, const T* __restrict__ beta, float eps) {
    __shared__ float red[32];
    const T* xr = X + (long long)blockIdx.x * ldx;
    T* yr = Y + (long long)blockIdx.x * ldy;
    const int tpr = blockDim.x;
    if (NORM == KF_NORM_SOFTMAX) {
        float m = -INFINITY;
        for (long long n = threadIdx.x; n < N; n += tpr) m = fmaxf(m, Elem<T>::load(xr + n));
        m = group_reduce<true>(m, tpr, red);
        float s = 0.f;
        for (long long n = threadIdx.x; n < N; n += tpr) s += exp2f((Elem<T>::load(xr + n) - m) * kLog2e);
        s = group_reduce<false>(s, tpr, red);
        const float inv = 1.0f / s;
        for (long long n = threadIdx.x; n < N; n += tpr)
            Elem<T>::store(yr + n, exp2f((Elem<T>::load(xr + n) - m) * kLog2e) * inv);
    } else {
        float mean = 0.f;
        if (NORM == KF_NORM_LAYERNORM) {
            float s = 0.f;
            for (long long n = threadIdx.x; n < N; n += tpr) s += Elem<T>::load(xr + n);
            mean = group_reduce<false>(s, tpr, red) / (float)N;
        }
        float q = 0.f;
        for (long long n = threadIdx.x; n < N; n += tpr) {
            const float d = Elem<T>::load(xr + n) - mean;
            q = fmaf(d, d, q);
        }
        q = group_reduce<false>(q, tpr, red);
        const float rstd = rsqrtf(q / (float)N + eps);
        for (long long n = threadIdx.x; n < N; n += tpr) {
            float o = (Elem<T>::load(xr + n) - mean) * rstd;
            if (gamma) o *= Elem<T>::load(gamma + n);
            if (beta && NORM == KF_NORM_LAYERNORM) o += Elem<T>::load(beta + n);
            Elem<T>::store(yr + n, o);
        }
    }
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <typename T, int NORM>
cudaError_t launch_typed(const void* X, long long ldx, void* Y, long long ldy, long long M, long long N,
                         const RowNormParams& rn, cudaStream_t st) {
    constexpr int E = Elem<T>::kVec;
    const T* x = static_cast<const T*>(X);
    T* y = static_cast<T*>(Y);
    const T* g = static_cast<const T*>(rn.gamma);
    const T* b = static_cast<const T*>(rn.beta);
    const long long NV = N / E;
    const bool vec_ok = (N % E == 0) && aligned16(X) && aligned16(Y) && (ldx % E == 0) && (ldy % E == 0) &&
                        (!g || aligned16(g)) && (!b || aligned16(b)) && NV <= 16 * 512 && N < (1ll << 30);
    if (!vec_ok) {
        for (long long r0 = 0; r0 < M; r0 += 1 << 30) {         // grid.x limit is 2^31-1
            const long long rows = (M - r0 < (1ll << 30)) ? M - r0 : (1ll << 30);
            row_norm_generic_kernel<T, NORM><<<(unsigned)rows, kRowThreads, 0, st>>>(
                x + r0 * ldx, ldx, y + r0 * ldy, ldy, N, g, b, rn.eps);
        }
        return cudaGetLastError();
    }
    // threads per row / vectors per thread: one warp per row while a row fits 16 vectors a lane
    int tpr = 32;
    if (NV > 32 * 16) { tpr = 64; while (tpr < 512 && (long long)tpr * 8 < NV) tpr <<= 1; }
    static const int env_tpr = [] {                              // sweep hook, read once
        const char* e = std::getenv("KF_ROW_TPR");
        return e ? std::atoi(e) : 0;
    }();
    if (env_tpr >= 32 && env_tpr <= 512 && (env_tpr & (env_tpr - 1)) == 0 && (long long)env_tpr * 16 >= NV)
        tpr = env_tpr;
    const int need = (int)((NV + tpr - 1) / tpr);
    int vpt = 1;
    while (vpt < need) vpt <<= 1;
    const int threads = tpr > kRowThreads ? tpr : kRowThreads;
    const int rows_per_cta = threads / tpr;
    const long long ctas = (M + rows_per_cta - 1) / rows_per_cta;
    if (ctas > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
#define KF_ROW_LAUNCH(V)                                                                               \
    row_norm_reg_kernel<T, NORM, V><<<(unsigned)ctas, threads, 0, st>>>(x, ldx, y, ldy, M, (int)N, tpr, g, b, \
                                                                       rn.eps)
    switch (vpt) {
    case 1: KF_ROW_LAUNCH(1); break;
    case 2: KF_ROW_LAUNCH(2); break;
    case 4: KF_ROW_LAUNCH(4); break;
    case 8: KF_ROW_LAUNCH(8); break;
    default: KF_ROW_LAUNCH(16); break;
    }
#undef KF_ROW_LAUNCH
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_dt(const void* X, long long ldx, void* Y, long long ldy, long long M, long long N,
                      const RowNormParams& rn, cudaStream_t st) {
    switch (rn.norm) {
    case KF_NORM_SOFTMAX: return launch_typed<T, KF_NORM_SOFTMAX>(X, ldx, Y, ldy, M, N, rn, st);
    case KF_NORM_LAYERNORM: return launch_typed<T, KF_NORM_LAYERNORM>(X, ldx, Y, ldy, M, N, rn, st);
    case KF_NORM_RMSNORM: return launch_typed<T, KF_NORM_RMSNORM>(X, ldx, Y, ldy, M, N, rn, st);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace

cudaError_t launch_row_norm(const void* X, long long ldx, void* Y, long long ldy, long long M, long long N,
                            int dt, const RowNormParams& rn, cudaStream_t st) {
    if (dt == KF_F32) return launch_dt<float>(X, ldx, Y, ldy, M, N, rn, st);
    return launch_dt<__nv_bfloat16>(X, ldx, Y, ldy, M, N, rn, st);
}

}  // namespace kf
