// bf16 linear + epilogue (+ split-N row-norm) on the Blackwell tensor cores: tcgen05.mma with the
// accumulator in TMEM, operands staged by TMA into 128B-swizzled shared memory, written for
// sm_100a only.
//
// One persistent CTA per SM walks output tiles of BM x BN = 128 x 256 (row-block major, so the
// N-tiles of one row block run side by side).  Warp roles:
//   warp 0      TMA producer: X tile [128 x 64] and W tile [256 x 64] per k-block into a 4-stage ring
//   warp 1      allocates TMEM (512 columns = two accumulators) and issues tcgen05.mma
//   warps 2..5  epilogue: tcgen05.ld (one thread = one output row), bias / activation / scale /
//               residual in fp32, per-row partial statistics of the tile, bf16 pack, swizzled
//               shared-memory staging, TMA store
// The two TMEM accumulators let the epilogue of tile i overlap the main loop of tile i+1.
//
// Row-norm (split-N): a row of N outputs spans N/256 tiles owned by different CTAs.  The epilogue
// sweeps its accumulator twice: sweep 1 applies the element-wise epilogue, gathers the tile's
// per-row statistics and writes the values back into TMEM (tcgen05.st); sweep 2 turns them into a
// 16-bit intermediate stored in Y -- softmax: bf16 exp(a - tile max); LayerNorm / RMSNorm: fp16
// (a - tile shift) * 2^-e with a per-row, per-tile power-of-two block scale, so the intermediate
// carries 11 significant bits relative to the largest deviation of the tile row.  The per-row
// partial {shift or max, sum, sum of squares, 2^e} goes to the workspace; the finishing kernel
// merges the partials of a row (online-softmax rescaling / Chan's merge) and rescales in place.
//
// Every wait on an mbarrier is bounded: when it gives up it records KF_ERR_TIMEOUT in the
// workspace status word, raises a CTA-wide abort flag and the CTA drains and exits.
#include <cuda.h>
#include <cuda_fp16.h>

#include <cstdlib>
#include <cstring>
#include <mutex>

#include "kf_tc.cuh"

namespace kf {
namespace {

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16;
constexpr int kStages = 4;
constexpr int kEpiWarps = 4;
constexpr int kThreads = 32 * (2 + kEpiWarps);
constexpr int kTmemCols = 512;                         // two fp32 accumulators of BN columns
constexpr uint32_t kABytes = BM * BK * 2;              // 16 KiB
constexpr uint32_t kBBytes = BN * BK * 2;              // 32 KiB
constexpr uint32_t kStageBytes = kABytes + kBBytes;
constexpr uint32_t kStoreBoxCols = 64, kStoreBoxRows = 32;
constexpr uint32_t kStageOutBytes = kStoreBoxCols * kStoreBoxRows * 2;   // 4 KiB per staging buffer
constexpr uint32_t kSmemA = 0;
constexpr uint32_t kSmemB = kSmemA + kStages * kABytes;
constexpr uint32_t kSmemOut = kSmemB + kStages * kBBytes;                 // 2 buffers per epilogue warp
constexpr uint32_t kSmemBar = kSmemOut + kEpiWarps * 2 * kStageOutBytes;
constexpr uint32_t kNumBars = 2 * kStages + 4;
constexpr uint32_t kSmemTmemPtr = kSmemBar + kNumBars * 8;
constexpr uint32_t kSmemAbort = kSmemTmemPtr + 4;
constexpr uint32_t kSmemTotal = kSmemAbort + 4;
constexpr uint32_t kSmemAlloc = kSmemTotal + 1024;     // slack to align the base to 1024 bytes
static_assert(kSmemAlloc <= 232448, "exceeds the 227 KiB per-CTA shared memory of sm_100");

constexpr long long kTimeoutCycles = 3000000000ll;     // about 1.5-2 s: far above any legitimate wait

// ---- PTX wrappers ----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}

// bounded wait: false = gave up (status recorded, abort raised) or another role aborted
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                            uint32_t* status, uint32_t code) {
    const long long t0 = clock64();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3F) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > kTimeoutCycles) {
                *abort_flag = 1;
                if (atomicCAS(status, 0u, (uint32_t)KF_ERR_TIMEOUT) == 0u) status[1] = code;
                __threadfence();
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* status, uint32_t code) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, status, code);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map), "r"(src),
                 "r"(c0), "r"(c1)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void tma_store_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N> __device__ __forceinline__ void tma_store_wait_all() {
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread i of the warp receives TMEM lane (base lane + i)
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
          "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
          "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void unpack_f16x8(const uint4& v, float* f) {
    const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 t = __half22float2(h[i]);
        f[2 * i] = t.x;
        f[2 * i + 1] = t.y;
    }
}

// shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 64 bf16 (128 B),
// 8-row groups 1024 B apart; `addr` is the shared address of the (1024-aligned) tile plus the
// byte offset of the k-slice inside the swizzle atom
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(1024u >> 4) << 32;      // stride between 8-row groups
    d |= (uint64_t)1 << 46;                 // descriptor version of sm_100
    d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
    return d;
}
// instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = 256
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

struct TcParams {
    int M, N, K;
    int tiles_m, tiles_n;
    const __nv_bfloat16* bias;
    const __nv_bfloat16* residual;
    long long ldr;
    int act;
    float scale;
    int norm;
    float4* partials;           // [tiles_m][tiles_n][128] when norm != NONE
    uint32_t* status;
};

// element-wise epilogue on 32 consecutive columns of one row (fast-math forms: bf16 output)
// (col0 .. col0+31 of the row; vectors of 8 columns at or beyond N are not read)
__device__ __forceinline__ void epilogue32(float (&a)[32], const TcParams& p, long long row, int col0, bool row_ok) {
    const int left = p.N - col0;
    if (p.bias) {
        const uint4* bp = reinterpret_cast<const uint4*>(p.bias + col0);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float b[8];
            if (q * 8 >= left) break;
            unpack<__nv_bfloat16>(__ldg(bp + q), b);
#pragma unroll
            for (int e = 0; e < 8; ++e) a[q * 8 + e] += b[e];
        }
    }
    if (p.act != KF_ACT_NONE) {
        switch (p.act) {
        case KF_ACT_GELU_ERF:
#pragma unroll
            for (int e = 0; e < 32; ++e) a[e] = apply_act<false>(KF_ACT_GELU_ERF, a[e]);
            break;
        case KF_ACT_GELU_TANH:
#pragma unroll
            for (int e = 0; e < 32; ++e) a[e] = apply_act<false>(KF_ACT_GELU_TANH, a[e]);
            break;
        case KF_ACT_SILU:
#pragma unroll
            for (int e = 0; e < 32; ++e) a[e] = apply_act<false>(KF_ACT_SILU, a[e]);
            break;
        case KF_ACT_RELU:
#pragma unroll
            for (int e = 0; e < 32; ++e) a[e] = fmaxf(a[e], 0.f);
            break;
        default:
#pragma unroll
            for (int e = 0; e < 32; ++e) a[e] = apply_act<false>(KF_ACT_SIGMOID, a[e]);
            break;
        }
    }
    if (p.scale != 1.0f) {
#pragma unroll
        for (int e = 0; e < 32; ++e) a[e] *= p.scale;
    }
    if (p.residual && row_ok) {
        const uint4* rp = reinterpret_cast<const uint4*>(p.residual + row * p.ldr + col0);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float r[8];
            if (q * 8 >= left) break;
            unpack<__nv_bfloat16>(__ldg(rp + q), r);
#pragma unroll
            for (int e = 0; e < 8; ++e) a[q * 8 + e] += r[e];
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1)
tc_linear_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                 const __grid_constant__ CUtensorMap tmY, const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* gbase = smem_raw + (base - raw);

    const uint32_t bar0 = base + kSmemBar;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kStages + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kStages + 2 + a); };
    volatile uint32_t* tmem_ptr = reinterpret_cast<volatile uint32_t*>(gbase + kSmemTmemPtr);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(gbase + kSmemAbort);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_tiles = p.tiles_m * p.tiles_n;
    const int kblocks = (p.K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), kEpiWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + kSmemTmemPtr),
                     "r"((uint32_t)kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int mb = tile / p.tiles_n, nb = tile % p.tiles_n;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 0x100u + stage)) { ok = false; break; }
                    mbar_arrive_expect_tx(full_bar(stage), kStageBytes);
                    tma_load_2d(base + kSmemA + stage * kABytes, &tmX, full_bar(stage), kb * BK, mb * BM);
                    tma_load_2d(base + kSmemB + stage * kBBytes, &tmW, full_bar(stage), kb * BK, nb * BN);
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status, 0x200u + acc)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status, 0x300u + stage)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = base + kSmemA + stage * kABytes;
                    const uint32_t b_addr = base + kSmemB + stage * kBBytes;
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        const uint64_t ad = smem_desc_sw128(a_addr + k * UMMA_K * 2);
                        const uint64_t bd = smem_desc_sw128(b_addr + k * UMMA_K * 2);
                        tc_mma_bf16(d_tmem, ad, bd, kIdesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    tc_commit(empty_bar(stage));          // stage reusable once these MMAs have read it
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit(tfull_bar(acc));                // accumulator complete
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int q = warp & 3;                            // TMEM lane quarter this warp may read
        const int ew = warp - 2;
        const uint32_t out0 = base + kSmemOut + ew * 2 * kStageOutBytes;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
            const int mb = tile / p.tiles_n, nb = tile % p.tiles_n;
            const int m0 = mb * BM, n0 = nb * BN;
            const long long row = (long long)m0 + q * 32 + lane;
            const bool row_ok = row < p.M;
            const int ncols = min(BN, p.N - n0);           // valid columns of this tile (multiple of 8)
            if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status, 0x400u + acc)) { ok = false; break; }
            tc_fence_after();
            const uint32_t t_row = tmem_base + acc * BN + ((uint32_t)(q * 32) << 16);

            // per-row partial statistics of this tile
            float st_shift = 0.f, st_s1 = 0.f, st_s2 = 0.f, st_scale = 1.f, mult = 1.f;
            if (p.norm != KF_NORM_NONE) {
                // sweep 1: epilogue values, statistics, values written back over the accumulator
                float mx = -INFINITY, amax = 0.f;
                for (int c = 0; c < BN / 32; ++c) {
                    if (c * 32 >= ncols) break;
                    uint32_t v[32];
                    tc_ld32(t_row + c * 32, v);
                    float a[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) a[e] = __uint_as_float(v[e]);
                    epilogue32(a, p, row, n0 + c * 32, row_ok);
                    if (p.norm == KF_NORM_SOFTMAX) {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (c * 32 + e < ncols) mx = fmaxf(mx, a[e]);
                    } else {
                        if (p.norm == KF_NORM_LAYERNORM) {
                            if (c == 0) st_shift = a[0];
#pragma unroll
                            for (int e = 0; e < 32; ++e) a[e] -= st_shift;
                        }
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (c * 32 + e < ncols) {
                                st_s1 += a[e];
                                st_s2 = fmaf(a[e], a[e], st_s2);
                                amax = fmaxf(amax, fabsf(a[e]));
                            }
                    }
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(a[e]);
                    tc_st32(t_row + c * 32, v);
                }
                if (p.norm == KF_NORM_SOFTMAX) {
                    st_shift = mx;
                } else {
                    // power-of-two block scale: stored fp16 values lie in (-2, 2)
                    uint32_t eb = (__float_as_uint(amax) >> 23) & 0xFFu;
                    eb = min(max(eb, 1u), 253u);
                    st_scale = __uint_as_float(eb << 23);
                    mult = __uint_as_float((254u - eb) << 23);
                }
            }
            for (int g = 0; g < BN / 64; ++g) {
                if (g * 64 >= ncols) break;
                const uint32_t buf = out0 + (g & 1) * kStageOutBytes;
                if (lane == 0) tma_store_wait_read<1>();   // the store that last read `buf` is done with it
                __syncwarp();
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int c0 = g * 64 + h * 32;
                    uint32_t v[32];
                    tc_ld32(t_row + c0, v);
                    float a[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) a[e] = __uint_as_float(v[e]);
                    uint32_t w[16];
                    if (p.norm == KF_NORM_NONE) {
                        epilogue32(a, p, row, n0 + c0, row_ok);
#pragma unroll
                        for (int e = 0; e < 16; ++e) w[e] = pack_bf16(a[2 * e], a[2 * e + 1]);
                    } else if (p.norm == KF_NORM_SOFTMAX) {
                        const float ms = st_shift * kLog2e;
#pragma unroll
                        for (int e = 0; e < 32; ++e) {
                            a[e] = exp2f(fmaf(a[e], kLog2e, -ms));
                            if (c0 + e < ncols) st_s1 += a[e];
                        }
#pragma unroll
                        for (int e = 0; e < 16; ++e) w[e] = pack_bf16(a[2 * e], a[2 * e + 1]);
                    } else {
#pragma unroll
                        for (int e = 0; e < 16; ++e) w[e] = pack_f16(a[2 * e] * mult, a[2 * e + 1] * mult);
                    }
                    // stage with the 128-byte swizzle the store map expects
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint32_t chunk = (uint32_t)(h * 4 + c) ^ (uint32_t)(lane & 7);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(buf + lane * 128u + chunk * 16u),
                                     "r"(w[c * 4 + 0]), "r"(w[c * 4 + 1]), "r"(w[c * 4 + 2]), "r"(w[c * 4 + 3])
                                     : "memory");
                    }
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0 && m0 + q * 32 < p.M) {
                    tma_store_2d(&tmY, buf, n0 + g * 64, m0 + q * 32);
                    tma_store_commit();
                }
            }
            // all TMEM accesses of this accumulator are done: hand it back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));
            if (p.norm != KF_NORM_NONE && row_ok)
                p.partials[((size_t)mb * p.tiles_n + nb) * BM + q * 32 + lane] =
                    make_float4(st_shift, st_s1, st_s2, st_scale);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) tma_store_wait_all<0>();
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (*abort_flag) {
            // give copies and MMAs in flight a bounded time to land before TMEM goes away
            for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        }
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols)
                     : "memory");
    }
}

// ------------------------------------------------------------------------------ finishing kernel
// One CTA per row: merge the row's per-tile partials, then rescale the bf16 intermediates in place.
constexpr int kFinThreads = 256;

__device__ __forceinline__ float block_sum(float v, float* red) {
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = 0.f;
    for (int i = 0; i < kFinThreads / 32; ++i) t += red[i];
    return t;
}
__device__ __forceinline__ float block_max(float v, float* red) {
    v = warp_max(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = red[0];
    for (int i = 1; i < kFinThreads / 32; ++i) t = fmaxf(t, red[i]);
    return t;
}

__global__ void __launch_bounds__(kFinThreads)
tc_rownorm_finish_kernel(__nv_bfloat16* Y, long long ldy, int N, int tiles_n, const float4* __restrict__ partials,
                         int norm, const __nv_bfloat16* __restrict__ gamma, const __nv_bfloat16* __restrict__ beta,
                         float eps) {
    extern __shared__ float tile_coef[];        // per tile: softmax factor / LayerNorm offset, then block scales
    float* tile_scale = tile_coef + tiles_n;
    __shared__ float red[kFinThreads / 32];
    const long long row = blockIdx.x;
    const int mb = (int)(row / BM), r = (int)(row % BM);
    const float4* pr = partials + ((size_t)mb * tiles_n) * BM + r;
    const int t = threadIdx.x;
    float rstd = 1.f;

    if (norm == KF_NORM_SOFTMAX) {
        float m = -INFINITY;
        for (int nb = t; nb < tiles_n; nb += kFinThreads) m = fmaxf(m, pr[(size_t)nb * BM].x);
        m = block_max(m, red);
        float l = 0.f;
        for (int nb = t; nb < tiles_n; nb += kFinThreads) {
            const float4 q = pr[(size_t)nb * BM];
            const float f = exp2f((q.x - m) * kLog2e);
            tile_coef[nb] = f;
            l = fmaf(q.y, f, l);
        }
        l = block_sum(l, red);
        rstd = 1.0f / l;                         // common factor; tile_coef holds exp(m_t - m)
    } else if (norm == KF_NORM_LAYERNORM) {
        float s = 0.f;
        for (int nb = t; nb < tiles_n; nb += kFinThreads) {
            const float4 q = pr[(size_t)nb * BM];
            const float cnt = (float)min(BN, N - nb * BN);
            s += q.x * cnt + q.y;                // sum of a over the tile = shift * count + sum(a - shift)
        }
        const float mean = block_sum(s, red) / (float)N;
        float m2 = 0.f;
        for (int nb = t; nb < tiles_n; nb += kFinThreads) {
            const float4 q = pr[(size_t)nb * BM];
            const float cnt = (float)min(BN, N - nb * BN);
            const float dmean = q.y / cnt;                       // tile mean minus tile shift
            const float m2_t = fmaxf(q.z - q.y * dmean, 0.f);    // centred sum of squares of the tile
            const float d = q.x + dmean - mean;
            m2 += fmaf(cnt * d, d, m2_t);                        // Chan's merge
            tile_coef[nb] = q.x - mean;
            tile_scale[nb] = q.w;
        }
        m2 = block_sum(m2, red);
        rstd = rsqrtf(m2 / (float)N + eps);
    } else {
        float s = 0.f;
        for (int nb = t; nb < tiles_n; nb += kFinThreads) {
            const float4 q = pr[(size_t)nb * BM];
            s += q.z;
            tile_coef[nb] = 0.f;
            tile_scale[nb] = q.w;
        }
        s = block_sum(s, red);
        rstd = rsqrtf(s / (float)N + eps);
    }
    __syncthreads();

    uint4* yr = reinterpret_cast<uint4*>(Y + row * ldy);
    const uint4* gv = reinterpret_cast<const uint4*>(gamma);
    const uint4* bv = reinterpret_cast<const uint4*>(beta);
    const int NV = N / 8;
    for (int idx = t; idx < NV; idx += kFinThreads) {
        float f[8];
        const uint4 raw = yr[idx];
        const int nb = idx / (BN / 8);
        if (norm == KF_NORM_SOFTMAX) {
            unpack<__nv_bfloat16>(raw, f);
            const float c = tile_coef[nb] * rstd;
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] *= c;
        } else {
            unpack_f16x8(raw, f);
            const float off = tile_coef[nb], sc = tile_scale[nb];
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] *= sc;
            float g[8], b[8];
            if (gamma) unpack<__nv_bfloat16>(__ldg(gv + idx), g);
            if (beta && norm == KF_NORM_LAYERNORM) unpack<__nv_bfloat16>(__ldg(bv + idx), b);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                float o = (f[e] + off) * rstd;
                if (gamma) o *= g[e];
                if (beta && norm == KF_NORM_LAYERNORM) o += b[e];
                f[e] = o;
            }
        }
        yr[idx] = pack<__nv_bfloat16>(f);
    }
}

// ------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            f = nullptr;
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

// 2-D bf16 row-major tensor [rows, cols] with pitch ld (elements); box = [box_rows, box_cols]
bool make_map(CUtensorMap* m, const void* ptr, long long rows, long long cols, long long ld, uint32_t box_cols,
              uint32_t box_rows, CUtensorMapL2promotion promo) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, promo,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
    static int n = [] {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 148;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
        return v;
    }();
    return n;
}

}  // namespace

// ---- built-in scratch for the allocation-free entry point -----------------------------------------
// Status block + per-row partial statistics for up to kStaticMaxTiles output tiles (4 MiB + 256 B).
// Every device that loads this library carries the array until the process exits.  In host code
// the name below is only a handle for cudaGetSymbolAddress; kernels receive the device address.
constexpr size_t kStaticMaxTiles = 2048;
constexpr size_t kStaticScratchBytes = kStatusBytes + kStaticMaxTiles * BM * sizeof(float4);
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

size_t tc_static_scratch_bytes() { return kStaticScratchBytes; }

kf_status tc_static_scratch(void** ptr) {
    static std::mutex mu;
    static void* cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return KF_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!cached[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return KF_ERR_CUDA;
        cached[dev] = p;
    }
    *ptr = cached[dev];
    return KF_OK;
}

static cudaEvent_t g_split_event = nullptr;
void tc_set_split_event(cudaEvent_t ev) { g_split_event = ev; }

void tc_tile_shape(int* bm, int* bn, int* bk, int* stages, int* epi_warps) {
    *bm = BM; *bn = BN; *bk = BK; *stages = kStages; *epi_warps = kEpiWarps;
}

size_t tc_partials_bytes(long long M, long long N) {
    const long long tm = (M + BM - 1) / BM, tn = (N + BN - 1) / BN;
    return (size_t)tm * tn * BM * sizeof(float4);
}

int tc_default_grid(long long M, long long N) {
    const long long tiles = ((M + BM - 1) / BM) * ((N + BN - 1) / BN);
    const int sms = sm_count();
    return (int)(tiles < sms ? tiles : sms);
}

kf_status launch_tc_linear(const void* X, long long ldx, const void* W, long long ldw, void* Y, long long ldy,
                           long long M, long long N, long long K, const EpilogueParams& ep, const RowNormParams& rn,
                           void* ws, int grid_override, cudaStream_t st, int* grid_out) {
    {   // opt in to the large dynamic shared memory once per device
        static std::mutex mu;
        static bool done[64] = {};
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return KF_ERR_CUDA;
        std::lock_guard<std::mutex> lock(mu);
        if (!done[dev]) {
            if (cudaFuncSetAttribute(tc_linear_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)kSmemAlloc) != cudaSuccess)
                return KF_ERR_CUDA;
            done[dev] = true;
        }
    }

    CUtensorMap tmX, tmW, tmY;
    if (!make_map(&tmX, X, M, K, ldx, BK, BM, CU_TENSOR_MAP_L2_PROMOTION_L2_256B) ||
        !make_map(&tmW, W, N, K, ldw, BK, BN, CU_TENSOR_MAP_L2_PROMOTION_L2_256B) ||
        !make_map(&tmY, Y, M, N, ldy, kStoreBoxCols, kStoreBoxRows, CU_TENSOR_MAP_L2_PROMOTION_NONE))
        return KF_ERR_CUDA;

    TcParams p;
    p.M = (int)M; p.N = (int)N; p.K = (int)K;
    p.tiles_m = (int)((M + BM - 1) / BM);
    p.tiles_n = (int)((N + BN - 1) / BN);
    p.bias = static_cast<const __nv_bfloat16*>(ep.bias);
    p.residual = static_cast<const __nv_bfloat16*>(ep.residual);
    p.ldr = ep.ldr;
    p.act = ep.act;
    p.scale = ep.scale;
    p.norm = rn.norm;
    p.partials = reinterpret_cast<float4*>(static_cast<uint8_t*>(ws) + kStatusBytes);
    p.status = static_cast<uint32_t*>(ws);

    int grid = tc_default_grid(M, N);
    if (grid_override > 0 && grid_override < grid) grid = grid_override;
    if (grid_out) *grid_out = grid;
    tc_linear_kernel<<<grid, kThreads, kSmemAlloc, st>>>(tmX, tmW, tmY, p);
    if (cudaGetLastError() != cudaSuccess) return KF_ERR_CUDA;
    if (g_split_event && cudaEventRecord(g_split_event, st) != cudaSuccess) return KF_ERR_CUDA;

    if (rn.norm != KF_NORM_NONE) {
        const size_t sm = (size_t)p.tiles_n * 2 * sizeof(float);
        tc_rownorm_finish_kernel<<<(unsigned)M, kFinThreads, sm, st>>>(
            static_cast<__nv_bfloat16*>(Y), ldy, (int)N, p.tiles_n, p.partials, rn.norm,
            static_cast<const __nv_bfloat16*>(rn.gamma), static_cast<const __nv_bfloat16*>(rn.beta), rn.eps);
        if (cudaGetLastError() != cudaSuccess) return KF_ERR_CUDA;
    }
    return KF_OK;
}

}  // namespace kf
