// fp32 linear + epilogue on the tensor cores by error-compensated TF32 splitting ("3xTF32").
//
// A single-pass TF32 product keeps 10 mantissa bits and misses the 1e-4 absolute gate of the fp32
// calls.  Here every operand is split once into hi = tf32(x) and lo = tf32(x - hi) (a pre-pass into
// the workspace), and each k-step issues three tcgen05.mma.kind::tf32 instructions into the same
// fp32 accumulator: lo*hi + hi*lo + hi*hi.  The dropped lo*lo term is below 2^-22 of the product, so
// the result is as good as an fp32 FMA chain, at a third of the TF32 rate.
//
// Same skeleton as the bf16 kernel: persistent CTA pairs (cta_group::2, 256 x 256 of Y per pair),
// warp 0 = TMA producer (four tiles per stage: X hi/lo, W hi/lo; 64 KiB per stage, 3 stages), warp 1 =
// TMEM allocator + MMA issuer, warps 2..9 = epilogue (bias, accurate activation, scale, residual in
// fp32; 128-byte row segments stored from registers; K in chunks of 512 whose sums are added in fp32
// through Y, because the tensor core's own accumulation truncates).  A row-norm, if any, runs afterwards as the
// in-place fp32 row kernel: the pre-norm row is held in fp32, so nothing is lost by not fusing it.
// Every mbarrier wait is bounded and reports through the workspace status word.
#include <cstdlib>
#include <mutex>

#include "kf_tc.cuh"
#include "kf_tc_ptx.cuh"

namespace kf {
namespace {

constexpr int BM = 128, BN = 256, BK = 32;             // BK fp32 = 128 bytes = one swizzle row
constexpr int UMMA_K = 8;                              // tf32: 8 k per instruction = 32 bytes
constexpr int kStages = 3;
// The tensor core adds into its fp32 accumulator with truncation, so a long K builds up a bias toward
// zero that grows with the number of accumulation steps (measured: 3.4e-5 at K = 1028, 1.5e-4 at 4100,
// 5.8e-4 at 16400 on unit-scale outputs).  K is therefore cut into chunks of kChunkBlocks k-blocks;
// each chunk is accumulated from zero in TMEM and the chunk sums are added in fp32 (round to nearest)
// by the epilogue warps through Y itself, which keeps the bias at the level of one chunk for any K.
constexpr int kChunkBlocks = 16;                       // 16 x 32 = 512 k per chunk
constexpr int kEpiWarps = 8;
constexpr int kSub = BN / 2;
constexpr int kThreads = 32 * (2 + kEpiWarps);
constexpr int kTmemCols = 512;
constexpr uint32_t kTileBytes = 128 * 128;             // 128 rows x 128 bytes: every staged tile (16 KiB)
constexpr uint32_t kStageBytes = 4 * kTileBytes;       // X hi, X lo, W-half hi, W-half lo
constexpr uint32_t kSmemBias = kStages * kStageBytes;  // 192 KiB ring, then 2 x BN floats of bias
constexpr uint32_t kSmemBar = kSmemBias + 2 * BN * 4;
constexpr uint32_t kNumBars = 2 * kStages + 6;
constexpr uint32_t kSmemTmemPtr = kSmemBar + kNumBars * 8;
constexpr uint32_t kSmemAbort = kSmemTmemPtr + 8;
constexpr uint32_t kSmemAlloc = kSmemAbort + 16;
static_assert(kSmemAlloc <= 232448, "exceeds the 227 KiB per-CTA shared memory of sm_100");

// instruction descriptor: D fp32, A and B tf32 (format 2), both K-major, M = 256 (pair), N = 256
constexpr uint32_t kIdescTf32 =
    (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((BM * 2) >> 4) << 24);

__device__ __forceinline__ void tc_mma_tf32_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(kIdescTf32), "r"(accumulate)
        : "memory");
}

// ---- operand split -------------------------------------------------------------------------------
__device__ __forceinline__ float to_tf32(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}

// src [rows, cols] with pitch ld (cols % 4 == 0, 16-byte aligned) -> hi, lo packed [rows, cols]
__global__ void __launch_bounds__(256)
split_tf32_kernel(const float* __restrict__ src, long long ld, float* __restrict__ hi, float* __restrict__ lo,
                  long long rows, int cols) {
    const int vec_per_row = cols / 4;
    const long long total = rows * vec_per_row;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const long long r = i / vec_per_row;
        const int c = (int)(i - r * vec_per_row);
        const float4 v = __ldcs(reinterpret_cast<const float4*>(src + r * ld) + c);
        float4 h, l;
        h.x = to_tf32(v.x); h.y = to_tf32(v.y); h.z = to_tf32(v.z); h.w = to_tf32(v.w);
        l.x = to_tf32(v.x - h.x); l.y = to_tf32(v.y - h.y); l.z = to_tf32(v.z - h.z); l.w = to_tf32(v.w - h.w);
        reinterpret_cast<float4*>(hi + r * cols)[c] = h;
        reinterpret_cast<float4*>(lo + r * cols)[c] = l;
    }
}

struct Tc32Params {
    int M, N, K;
    int tiles_m, tiles_n;
    const float* bias;
    const float* residual;
    long long ldr;
    int act;
    float scale;
    float* Y;
    long long ldy;
    uint32_t* status;
    long long timeout_cycles;
};

// element-wise epilogue on 32 consecutive columns of one row, accurate fp32 forms
template <int ACT>
__device__ __forceinline__ void epilogue32_f32(float (&a)[32], const Tc32Params& p, const float* bias32, long long row,
                                               int col0, bool row_ok) {
    if (bias32) {
        const float4* bp = reinterpret_cast<const float4*>(bias32);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float4 b = bp[q];
            a[q * 4 + 0] += b.x; a[q * 4 + 1] += b.y; a[q * 4 + 2] += b.z; a[q * 4 + 3] += b.w;
        }
    }
    if (ACT != KF_ACT_NONE) {
#pragma unroll
        for (int e = 0; e < 32; ++e) a[e] = apply_act<true>(ACT, a[e]);
    }
    if (p.scale != 1.0f) {
#pragma unroll
        for (int e = 0; e < 32; ++e) a[e] *= p.scale;
    }
    if (p.residual && row_ok) {
        const int left = p.N - col0;
        const float4* rp = reinterpret_cast<const float4*>(p.residual + row * p.ldr + col0);
#pragma unroll
        for (int q = 0; q < 8; ++q)
            if (q * 4 < left) {
                const float4 r = __ldg(rp + q);
                a[q * 4 + 0] += r.x; a[q * 4 + 1] += r.y; a[q * 4 + 2] += r.z; a[q * 4 + 3] += r.w;
            }
    }
}

// ACT: the activation compiled in (the accurate forms are long; with all six behind a run-time switch in the
// unrolled epilogue the kernel spent five times its main loop fetching instructions)
template <int ACT>
__global__ void __launch_bounds__(kThreads, 1)
tc32_linear_kernel(const __grid_constant__ CUtensorMap tmXh, const __grid_constant__ CUtensorMap tmXl,
                   const __grid_constant__ CUtensorMap tmWh, const __grid_constant__ CUtensorMap tmWl,
                   const Tc32Params p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if (base & 1023u) {
        if (threadIdx.x == 0 && atomicCAS(p.status, 0u, (uint32_t)KF_ERR_CUDA) == 0u) p.status[1] = 0x901u;
        return;
    }
    const uint32_t rank = cluster_ctarank();             // rank 0 of a pair issues the MMAs
    const int unit = (int)(blockIdx.x >> 1), num_units = (int)(gridDim.x >> 1);
    const uint32_t bar0 = base + kSmemBar;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kStages + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kStages + 2 + a); };
    auto bias_bar = [&](int b) { return bar0 + 8u * (2 * kStages + 4 + b); };
    volatile uint32_t* tmem_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + kSmemTmemPtr);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem_raw + kSmemAbort);
    float* bias_smem = reinterpret_cast<float*>(smem_raw + kSmemBias);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int units_m = (p.tiles_m + 1) / 2;
    const int num_tiles = units_m * p.tiles_n;
    const int kblocks = (p.K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), kEpiWarps * 2);
            mbar_init(bias_bar(a), kEpiWarps);
        }
        *abort_flag = 0;
        *reinterpret_cast<volatile long long*>(smem_raw + kSmemAbort + 8) = p.timeout_cycles;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + kSmemTmemPtr),
                     "r"((uint32_t)kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int tile = unit; tile < num_tiles && ok; tile += num_units) {
                const int mb = (tile / p.tiles_n) * 2 + (int)rank, nb = tile % p.tiles_n;
                for (int kb = 0; kb < kblocks; ++kb) {             // chunks need nothing special here
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 0x110u + stage)) { ok = false; break; }
                    if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), 2 * kStageBytes);
                    const uint32_t lead_bar = map_to_cta(full_bar(stage), 0);
                    const uint32_t s0 = base + stage * kStageBytes;
                    const int wrow = nb * BN + (int)rank * 128;
                    tma_load_2d_pair(s0 + 0 * kTileBytes, &tmXh, lead_bar, kb * BK, mb * BM);
                    tma_load_2d_pair(s0 + 1 * kTileBytes, &tmXl, lead_bar, kb * BK, mb * BM);
                    tma_load_2d_pair(s0 + 2 * kTileBytes, &tmWh, lead_bar, kb * BK, wrow);
                    tma_load_2d_pair(s0 + 3 * kTileBytes, &tmWl, lead_bar, kb * BK, wrow);
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (pair leader)
        if (lane == 0 && rank == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = unit; tile < num_tiles && ok; tile += num_units) {
                for (int kb0 = 0; kb0 < kblocks && ok; kb0 += kChunkBlocks) {       // one accumulator per K chunk
                    if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status, 0x210u + acc)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + acc * BN;
                    const int kb1 = min(kblocks, kb0 + kChunkBlocks);
                    for (int kb = kb0; kb < kb1; ++kb) {
                        if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status, 0x310u + stage)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t s0 = base + stage * kStageBytes;
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K; ++k) {
                            const uint32_t off = k * UMMA_K * 4;
                            const uint64_t ah = smem_desc_sw128(s0 + 0 * kTileBytes + off);
                            const uint64_t al = smem_desc_sw128(s0 + 1 * kTileBytes + off);
                            const uint64_t bh = smem_desc_sw128(s0 + 2 * kTileBytes + off);
                            const uint64_t bl = smem_desc_sw128(s0 + 3 * kTileBytes + off);
                            tc_mma_tf32_pair(d_tmem, al, bh, (kb != kb0 || k != 0) ? 1u : 0u);     // small terms first
                            tc_mma_tf32_pair(d_tmem, ah, bl, 1u);
                            tc_mma_tf32_pair(d_tmem, ah, bh, 1u);
                        }
                        tc_commit_pair(empty_bar(stage));
                        tc_commit_pair(map_to_cta(empty_bar(stage), 1));
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                    if (!ok) break;
                    tc_commit_pair(tfull_bar(acc));
                    tc_commit_pair(map_to_cta(tfull_bar(acc), 1));
                    if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        const int et = threadIdx.x - 64;
        const int cb = half * kSub;
        uint32_t acc = 0, acc_phase = 0, it = 0;
        bool ok = true;
        for (int tile = unit; tile < num_tiles && ok; tile += num_units, ++it) {
            const int mb = (tile / p.tiles_n) * 2 + (int)rank, nb = tile % p.tiles_n;
            const int m0 = mb * BM, n0 = nb * BN;
            const long long row = (long long)m0 + q * 32 + lane;
            const bool row_ok = row < p.M;
            float* yrow = p.Y + row * p.ldy + n0 + cb;
            const int ncols = max(0, min(kSub, p.N - n0 - cb));     // multiple of 4
            const int nchunks = (ncols + 31) >> 5;

            float* bias_t = nullptr;
            if (p.bias) {                                   // staged once per tile, used by its last chunk
                bias_t = bias_smem + (it & 1u) * BN;
                bias_t[et] = (n0 + et < p.N) ? p.bias[n0 + et] : 0.f;
                __syncwarp();
                if (lane == 0) mbar_arrive(bias_bar(it & 1u));
                if (!mbar_wait(bias_bar(it & 1u), (it >> 1) & 1u, abort_flag, p.status, 0x510u)) { ok = false; break; }
                bias_t += cb;
            }
            for (int kb0 = 0; kb0 < kblocks && ok; kb0 += kChunkBlocks) {
                const bool first = kb0 == 0, last = kb0 + kChunkBlocks >= kblocks;
                if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status, 0x410u + acc)) { ok = false; break; }
                tc_fence_after();
                const uint32_t t_row = tmem_base + acc * BN + cb + ((uint32_t)(q * 32) << 16);
                uint32_t v[2][32];
                if (nchunks > 0) {
                    tc_ld32_issue(t_row, v[0]);
#pragma unroll
                    for (int c = 0; c < kSub / 32; ++c) {
                        if (c < nchunks) {
                            tc_ld_wait(v[c & 1]);
                            if (c + 1 < nchunks) tc_ld32_issue(t_row + (c + 1) * 32, v[(c + 1) & 1]);
                            float a[32];
#pragma unroll
                            for (int e = 0; e < 32; ++e) a[e] = __uint_as_float(v[c & 1][e]);
                            const int left = ncols - c * 32;
                            float4* d = reinterpret_cast<float4*>(yrow + c * 32);
                            if (!first && row_ok) {         // add the sum of the earlier chunks (this thread wrote it)
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    if (j * 4 < left) {
                                        const float4 prev = d[j];
                                        a[j * 4 + 0] += prev.x; a[j * 4 + 1] += prev.y;
                                        a[j * 4 + 2] += prev.z; a[j * 4 + 3] += prev.w;
                                    }
                            }
                            if (last) epilogue32_f32<ACT>(a, p, bias_t ? bias_t + c * 32 : nullptr, row, n0 + cb + c * 32, row_ok);
                            if (row_ok) {
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    if (j * 4 < left) d[j] = make_float4(a[j * 4], a[j * 4 + 1], a[j * 4 + 2], a[j * 4 + 3]);
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (rank != 0) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));
                    else mbar_arrive(tempty_bar(acc));
                }
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        if (*abort_flag) {
            for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        }
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols)
                     : "memory");
    }
}

// ------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn32() {
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

// packed fp32 [rows, cols]; box = 128 rows x 32 columns (128 bytes), 128-byte swizzle, zero fill
bool make_map32(CUtensorMap* m, const float* ptr, long long rows, long long cols) {
    EncodeTiledFn fn = encode_fn32();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
    cuuint32_t box[2] = {(cuuint32_t)BK, 128};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline size_t round256(size_t b) { return (b + 255) & ~(size_t)255; }

int sm_count32() {
    static int n = [] {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 148;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
        return v;
    }();
    return n;
}

}  // namespace

// bytes behind the status block: hi and lo copies of X [M,K] and W [N,K], each 256-byte aligned
size_t tc32_split_bytes(long long M, long long N, long long K) {
    return 2 * round256((size_t)M * K * 4) + 2 * round256((size_t)N * K * 4);
}

// shapes the 3xTF32 kernel serves: enough work to pay for the split.  A single row block (M <= 128) runs too:
// the second CTA of each pair then loads zero-filled rows and stores nothing, and half the MMA is idle, yet
// the call still beats the CUDA-core kernels several times over (64 x 2048 x 2048: 0.087 vs 0.885 ms)
bool tc32_shape_ok(long long M, long long N, long long K) {
    // three launches (two operand splits and the GEMM) cost about 0.03 ms; from about 6e7 flop on they beat the
    // CUDA-core kernels (300 x 520 x 200: 0.034 vs 0.057 ms; 1024^3: 0.067 vs 0.307 ms)
    static const double min_flops = [] {                   // KF_TC32_MIN_FLOPS moves the gate (sweeps)
        const char* e = std::getenv("KF_TC32_MIN_FLOPS");
        return e ? std::atof(e) : 6.0e7;
    }();
    return K >= 32 && K % 4 == 0 && N % 4 == 0 && 2.0 * (double)M * (double)N * (double)K >= min_flops;
}

int tc32_default_grid(long long M, long long N) {
    const long long tm = (M + BM - 1) / BM, tn = (N + BN - 1) / BN;
    const long long units = ((tm + 1) / 2) * tn;
    const long long slots = sm_count32() / 2;
    return (int)((units < slots ? units : slots) * 2);
}

namespace {
template <int ACT>
kf_status launch_tc32_instance(const cudaLaunchConfig_t& lc, const CUtensorMap& tmXh, const CUtensorMap& tmXl,
                               const CUtensorMap& tmWh, const CUtensorMap& tmWl, const Tc32Params& p) {
    auto kernel = tc32_linear_kernel<ACT>;
    {   // opt in to the large dynamic shared memory once per device
        static std::mutex mu;
        static bool done[64] = {};
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return KF_ERR_CUDA;
        std::lock_guard<std::mutex> lock(mu);
        if (!done[dev]) {
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemAlloc) != cudaSuccess)
                return KF_ERR_CUDA;
            done[dev] = true;
        }
    }
    if (cudaLaunchKernelEx(&lc, kernel, tmXh, tmXl, tmWh, tmWl, p) != cudaSuccess) {
        cudaGetLastError();
        return KF_ERR_CUDA;
    }
    return KF_OK;
}
}  // namespace

kf_status launch_tc32_linear(const void* X, long long ldx, const void* W, long long ldw, void* Y, long long ldy,
                             long long M, long long N, long long K, const EpilogueParams& ep, void* ws,
                             cudaStream_t st, int* grid_out) {
    uint8_t* cur = static_cast<uint8_t*>(ws) + kStatusBytes;
    float* Xh = reinterpret_cast<float*>(cur); cur += round256((size_t)M * K * 4);
    float* Xl = reinterpret_cast<float*>(cur); cur += round256((size_t)M * K * 4);
    float* Wh = reinterpret_cast<float*>(cur); cur += round256((size_t)N * K * 4);
    float* Wl = reinterpret_cast<float*>(cur);

    const int split_grid = sm_count32() * 8;
    split_tf32_kernel<<<split_grid, 256, 0, st>>>(static_cast<const float*>(X), ldx, Xh, Xl, M, (int)K);
    split_tf32_kernel<<<split_grid, 256, 0, st>>>(static_cast<const float*>(W), ldw, Wh, Wl, N, (int)K);
    if (cudaGetLastError() != cudaSuccess) return KF_ERR_CUDA;

    CUtensorMap tmXh, tmXl, tmWh, tmWl;
    if (!make_map32(&tmXh, Xh, M, K) || !make_map32(&tmXl, Xl, M, K) || !make_map32(&tmWh, Wh, N, K) ||
        !make_map32(&tmWl, Wl, N, K))
        return KF_ERR_CUDA;

    Tc32Params p;
    p.M = (int)M; p.N = (int)N; p.K = (int)K;
    p.tiles_m = (int)((M + BM - 1) / BM);
    p.tiles_n = (int)((N + BN - 1) / BN);
    p.bias = static_cast<const float*>(ep.bias);
    p.residual = static_cast<const float*>(ep.residual);
    p.ldr = ep.ldr;
    p.act = ep.act;
    p.scale = ep.scale;
    p.Y = static_cast<float*>(Y);
    p.ldy = ldy;
    p.status = static_cast<uint32_t*>(ws);
    static const long long timeout_cycles = [] {
        const char* e = std::getenv("KF_TC_TIMEOUT_MS");
        const long long ms = e ? std::atoll(e) : 0;
        return ms > 0 ? ms * 2000000ll : kTimeoutCycles;
    }();
    p.timeout_cycles = timeout_cycles;

    const int grid = tc32_default_grid(M, N);
    if (grid_out) *grid_out = grid;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)grid);
    lc.blockDim = dim3(kThreads);
    lc.dynamicSmemBytes = kSmemAlloc;
    lc.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    lc.attrs = at;
    lc.numAttrs = 1;
    switch (ep.act) {
    case KF_ACT_NONE: return launch_tc32_instance<KF_ACT_NONE>(lc, tmXh, tmXl, tmWh, tmWl, p);
    case KF_ACT_GELU_ERF: return launch_tc32_instance<KF_ACT_GELU_ERF>(lc, tmXh, tmXl, tmWh, tmWl, p);
    case KF_ACT_GELU_TANH: return launch_tc32_instance<KF_ACT_GELU_TANH>(lc, tmXh, tmXl, tmWh, tmWl, p);
    case KF_ACT_SILU: return launch_tc32_instance<KF_ACT_SILU>(lc, tmXh, tmXl, tmWh, tmWl, p);
    case KF_ACT_RELU: return launch_tc32_instance<KF_ACT_RELU>(lc, tmXh, tmXl, tmWh, tmWl, p);
    case KF_ACT_SIGMOID: return launch_tc32_instance<KF_ACT_SIGMOID>(lc, tmXh, tmXl, tmWh, tmWl, p);
    default: return KF_ERR_INVALID_ARG;
    }
}

}  // namespace kf
