// bf16 linear + epilogue (+ split-N row-norm) on the Blackwell tensor cores: tcgen05.mma with the
// accumulator in TMEM, operands staged by TMA into 128B-swizzled shared memory, written for
// sm_100a only.
//
// One persistent CTA per SM walks output tiles of BM x BN = 128 x 256 (row-block major, so the
// N-tiles of one row block run side by side).  Warp roles:
//   warp 0      TMA producer: X tile [128 x 64] and W tile [256 x 64] per k-block into a 4-stage ring
//   warp 1      allocates TMEM (512 columns = two accumulators) and issues tcgen05.mma
//   warps 2..9  epilogue: two warps per TMEM lane quarter, 128 columns each; software-pipelined
//               tcgen05.ld (one thread = one output row), bias (staged as fp32 in shared memory) /
//               activation / scale / residual in fp32, per-row partial statistics of the 128-column
//               sub-tile, 16-bit pack, 64-byte row segments stored straight from registers (shared
//               memory is left to the operand ring: 6 stages of 32 KiB with CTA pairs; a seventh
//               stage measured no faster)
// The two TMEM accumulators let the epilogue of tile i overlap the main loop of tile i+1.
//
// Row-norm (split-N): a row of N outputs spans N/128 sub-tiles owned by different warps and CTAs.  The epilogue
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
#include "kf_tc_ptx.cuh"

namespace kf {
namespace {

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16;
constexpr int kMaxStages = 6;
constexpr int kEpiWarps = 8;                           // two per TMEM lane quarter, 128 columns each
constexpr int kSub = BN / 2;                           // columns per epilogue warp = statistics sub-tile
constexpr int kThreads = 32 * (2 + kEpiWarps);
constexpr int kTmemCols = 512;                         // two fp32 accumulators of BN columns
constexpr uint32_t kABytes = BM * BK * 2;              // 16 KiB
// CG = CTAs per MMA.  CG 1: a CTA stages the whole 256-row W tile (32 KiB, 4 stages).  CG 2: the two
// CTAs of a cluster stage 128 rows of W each (16 KiB, 6 stages) and one tcgen05.mma.cta_group::2
// of M = 256 reads both halves, which halves the shared-memory traffic per flop.
template <int CG> struct Cfg {
    static constexpr int kStages = CG == 2 ? 6 : 4;
    static constexpr uint32_t kBRows = BN / CG;
    static constexpr uint32_t kBBytes = kBRows * BK * 2;
    static constexpr uint32_t kStageBytes = kABytes + kBBytes;
    static constexpr uint32_t kSmemB = kStages * kABytes;
    static_assert(kStages * kStageBytes == 192 * 1024, "operand ring is 192 KiB in both modes");
};
constexpr uint32_t kSmemA = 0;
constexpr uint32_t kSmemBias = 192 * 1024;             // 2 x BN floats (double buffered), behind the operand ring
constexpr uint32_t kSmemBar = kSmemBias + 2 * BN * 4;
constexpr uint32_t kNumBars = 2 * kMaxStages + 6;         // ring full/empty, accumulator full/empty, bias ready
constexpr uint32_t kSmemTmemPtr = kSmemBar + kNumBars * 8;
constexpr uint32_t kSmemAbort = kSmemTmemPtr + 8;      // abort flag (4 B, 8-byte aligned), then the wait limit (8 B)
constexpr uint32_t kSmemAlloc = kSmemAbort + 16;
static_assert(kSmemAlloc <= 232448, "exceeds the 227 KiB per-CTA shared memory of sm_100");

// instruction descriptor: D fp32, A and B bf16, both K-major, M = 128 * CG, N = 256
template <int CG>
constexpr uint32_t kIdesc =
    (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((BM * CG) >> 4) << 24);

struct TcParams {
    int M, N, K;
    int tiles_m, tiles_n;
    int nsub;                   // statistics sub-tiles per row = ceil(N / 128)
    const __nv_bfloat16* bias;
    const __nv_bfloat16* residual;
    long long ldr;
    int act;
    float scale;
    int norm;
    float4* partials;           // [tiles_m * 128 rows][nsub] when norm != NONE
    uint32_t* status;
    __nv_bfloat16* Y;           // output (or 16-bit intermediate), row pitch ldy
    long long ldy;
    int debug;                  // timing experiments only (results are wrong): 1 no TMA loads, 2 no MMAs, 4 no epilogue work;
                                // 512 = the producer never signals, so every wait runs into its limit (time-out test)
    long long timeout_cycles;   // limit of every bounded wait
};

// element-wise epilogue on 32 consecutive columns of one row, fast-math forms (bf16 output).
// bias32: the 32 bias values as fp32 in shared memory (or nullptr); col0 = global column of a[0];
// 8-column vectors at or beyond N are not read from the residual.
__device__ __forceinline__ void epilogue32(float (&a)[32], const TcParams& p, const float* bias32, long long row,
                                           int col0, bool row_ok) {
    // the residual comes from global memory (often DRAM): issue its loads first, use them last
    const bool has_res = p.residual && row_ok && !(p.debug & 64);
    uint4 rv[4];
    if (has_res) {
        const int left = p.N - col0;
        const uint4* rp = reinterpret_cast<const uint4*>(p.residual + row * p.ldr + col0);
#pragma unroll
        for (int q = 0; q < 4; ++q) rv[q] = (q * 8 < left) ? __ldg(rp + q) : make_uint4(0, 0, 0, 0);
    }
    if (bias32) {
        const float4* bp = reinterpret_cast<const float4*>(bias32);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float4 b = bp[q];
            a[q * 4 + 0] += b.x; a[q * 4 + 1] += b.y; a[q * 4 + 2] += b.z; a[q * 4 + 3] += b.w;
        }
    }
    if (p.act != KF_ACT_NONE && !(p.debug & 32)) {
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
    if (has_res) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float r[8];
            unpack<__nv_bfloat16>(rv[q], r);
#pragma unroll
            for (int e = 0; e < 8; ++e) a[q * 8 + e] += r[e];
        }
    }
}

// one thread writes its 32 packed 16-bit values (64 contiguous bytes of its output row); 8-column
// vectors at or beyond the valid columns are skipped
__device__ __forceinline__ void store_row32(__nv_bfloat16* dst, const uint32_t (&w)[16], int valid_cols) {
    uint4* d = reinterpret_cast<uint4*>(dst);
#pragma unroll
    for (int j = 0; j < 4; ++j)
        if (j * 8 < valid_cols) d[j] = make_uint4(w[j * 4 + 0], w[j * 4 + 1], w[j * 4 + 2], w[j * 4 + 3]);
}

template <int CG>
__global__ void __launch_bounds__(kThreads, 1)
tc_linear_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, const TcParams p) {
    using C = Cfg<CG>;
    constexpr int kStages = C::kStages;
    constexpr uint32_t kSmemB = C::kSmemB, kBBytes = C::kBBytes;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if (base & 1023u) {                                 // swizzled tiles need a 1024-byte aligned base
        if (threadIdx.x == 0 && atomicCAS(p.status, 0u, (uint32_t)KF_ERR_CUDA) == 0u) p.status[1] = 0x900u;
        return;                                         // (same in both CTAs of a pair: the layout is identical)
    }
    const uint32_t rank = CG == 2 ? cluster_ctarank() : 0u;       // rank 0 of a pair issues the MMAs
    const int unit = CG == 2 ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int num_units = CG == 2 ? (int)(gridDim.x >> 1) : (int)gridDim.x;
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
    // a work unit is a BM*CG x BN block of the output: one tile, or the two row-adjacent tiles of a pair
    const int units_m = (p.tiles_m + CG - 1) / CG;
    const int num_tiles = units_m * p.tiles_n;
    const int kblocks = (p.K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), kEpiWarps * CG);   // the leader's collects the epilogue warps of both CTAs
            mbar_init(bias_bar(a), kEpiWarps);
        }
        *abort_flag = 0;
        *reinterpret_cast<volatile long long*>(smem_raw + kSmemAbort + 8) = p.timeout_cycles;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        if (CG == 2) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + kSmemTmemPtr),
                         "r"((uint32_t)kTmemCols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + kSmemTmemPtr),
                         "r"((uint32_t)kTmemCols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();                    // the peer's barriers exist before anyone signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int tile = unit; tile < num_tiles && ok; tile += num_units) {
                if (p.debug & 512) break;                  // time-out test: nothing is ever loaded or signalled
                const int mb = (tile / p.tiles_n) * CG + (int)rank, nb = tile % p.tiles_n;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 0x100u + stage)) { ok = false; break; }
                    if (p.debug & 1) {
                        if (rank == 0) mbar_arrive(full_bar(stage));
                    } else if (CG == 2) {
                        // both CTAs' copies complete on the leader's barrier, which expects the bytes of both
                        if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), 2 * C::kStageBytes);
                        const uint32_t lead_bar = map_to_cta(full_bar(stage), 0);
                        tma_load_2d_pair(base + kSmemA + stage * kABytes, &tmX, lead_bar, kb * BK, mb * BM);
                        tma_load_2d_pair(base + kSmemB + stage * kBBytes, &tmW, lead_bar, kb * BK,
                                         nb * BN + (int)(rank * C::kBRows));
                    } else {
                        mbar_arrive_expect_tx(full_bar(stage), C::kStageBytes);
                        tma_load_2d(base + kSmemA + stage * kABytes, &tmX, full_bar(stage), kb * BK, mb * BM);
                        tma_load_2d(base + kSmemB + stage * kBBytes, &tmW, full_bar(stage), kb * BK, nb * BN);
                    }
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && rank == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = unit; tile < num_tiles && ok; tile += num_units) {
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
                        if (p.debug & 2) break;
                        const uint64_t ad = smem_desc_sw128(a_addr + k * UMMA_K * 2);
                        const uint64_t bd = smem_desc_sw128(b_addr + k * UMMA_K * 2);
                        if (CG == 2) tc_mma_bf16_pair(d_tmem, ad, bd, kIdesc<2>, (kb | k) != 0 ? 1u : 0u);
                        else tc_mma_bf16(d_tmem, ad, bd, kIdesc<1>, (kb | k) != 0 ? 1u : 0u);
                    }
                    // stage reusable (in both CTAs of a pair) once these MMAs have read it
                    if (CG == 2) {
                        tc_commit_pair(empty_bar(stage));
                        tc_commit_pair(map_to_cta(empty_bar(stage), 1));
                    } else {
                        tc_commit(empty_bar(stage));
                    }
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                // accumulator complete: each CTA's epilogue reads its own 128 rows
                if (CG == 2) {
                    tc_commit_pair(tfull_bar(acc));
                    tc_commit_pair(map_to_cta(tfull_bar(acc), 1));
                } else {
                    tc_commit(tfull_bar(acc));
                }
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int q = warp & 3;                            // TMEM lane quarter this warp may access
        const int half = (warp - 2) >> 2;                  // which 128 columns of the tile
        const int et = threadIdx.x - 64;                   // 0..255 among the epilogue threads
        uint32_t acc = 0, acc_phase = 0, it = 0;
        bool ok = true;
        for (int tile = unit; tile < num_tiles && ok; tile += num_units, ++it) {
            const int mb = (tile / p.tiles_n) * CG + (int)rank, nb = tile % p.tiles_n;
            const int m0 = mb * BM, n0 = nb * BN;
            const int cb = half * kSub;                    // first tile column of this warp
            const long long row = (long long)m0 + q * 32 + lane;
            const bool row_ok = row < p.M;
            __nv_bfloat16* yrow = p.Y + row * p.ldy + n0 + cb;      // dereferenced only when row_ok
            const int ncols = max(0, min(kSub, p.N - n0 - cb));     // valid columns of this warp (multiple of 8)
            const int nchunks = (p.debug & 4) ? 0 : (ncols + 31) >> 5;

            // bias of the tile as fp32 in shared memory, double buffered across tiles
            float* bias_t = nullptr;
            if (p.bias) {
                bias_t = bias_smem + (it & 1u) * BN;
                bias_t[et] = (n0 + et < p.N) ? __bfloat162float(p.bias[n0 + et]) : 0.f;
                __syncwarp();
                if (lane == 0) mbar_arrive(bias_bar(it & 1u));        // release: this warp's 32 values are written
                if (!mbar_wait(bias_bar(it & 1u), (it >> 1) & 1u, abort_flag, p.status, 0x500u)) { ok = false; break; }
                bias_t += cb;
            }
            if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status, 0x400u + acc)) { ok = false; break; }
            tc_fence_after();
            const uint32_t t_row = tmem_base + acc * BN + cb + ((uint32_t)(q * 32) << 16);

            float st_shift = 0.f, st_s1 = 0.f, st_s2 = 0.f, st_scale = 1.f, mult = 1.f;
            uint32_t v[2][32];
            if (p.norm != KF_NORM_NONE && nchunks > 0) {
                // sweep 1: epilogue values, statistics (4 independent accumulators each), write-back to TMEM
                float s1[4] = {0.f, 0.f, 0.f, 0.f}, s2[4] = {0.f, 0.f, 0.f, 0.f};
                float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY}, am[4] = {0.f, 0.f, 0.f, 0.f};
                if (!(p.debug & 16)) tc_ld32_issue(t_row, v[0]);
#pragma unroll
                for (int c = 0; c < kSub / 32; ++c) {
                    if (c < nchunks) {
                        if (!(p.debug & 16)) {
                            tc_ld_wait(v[c & 1]);
                            if (c + 1 < nchunks) tc_ld32_issue(t_row + (c + 1) * 32, v[(c + 1) & 1]);
                        }
                        float a[32];
#pragma unroll
                        for (int e = 0; e < 32; ++e) a[e] = __uint_as_float(v[c & 1][e]);
                        epilogue32(a, p, bias_t ? bias_t + c * 32 : nullptr, row, n0 + cb + c * 32, row_ok);
                        const bool full = (c + 1) * 32 <= ncols;
                        if (p.norm == KF_NORM_SOFTMAX) {
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if (full || c * 32 + e < ncols) mx[e & 3] = fmaxf(mx[e & 3], a[e]);
                        } else {
                            if (p.norm == KF_NORM_LAYERNORM) {
                                if (c == 0) st_shift = a[0];
#pragma unroll
                                for (int e = 0; e < 32; ++e) a[e] -= st_shift;
                            }
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if (full || c * 32 + e < ncols) {
                                    s1[e & 3] += a[e];
                                    s2[e & 3] = fmaf(a[e], a[e], s2[e & 3]);
                                    am[e & 3] = fmaxf(am[e & 3], fabsf(a[e]));
                                }
                        }
                        uint32_t wb[32];
#pragma unroll
                        for (int e = 0; e < 32; ++e) wb[e] = __float_as_uint(a[e]);
                        if (!(p.debug & 16)) tc_st32(t_row + c * 32, wb);
                    }
                }
                tc_st_wait();
                if (p.norm == KF_NORM_SOFTMAX) {
                    st_shift = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                } else {
                    st_s1 = (s1[0] + s1[1]) + (s1[2] + s1[3]);
                    st_s2 = (s2[0] + s2[1]) + (s2[2] + s2[3]);
                    const float amax = fmaxf(fmaxf(am[0], am[1]), fmaxf(am[2], am[3]));
                    // power-of-two block scale: stored fp16 values lie in (-2, 2)
                    uint32_t eb = (__float_as_uint(amax) >> 23) & 0xFFu;
                    eb = min(max(eb, 1u), 253u);
                    st_scale = __uint_as_float(eb << 23);
                    mult = __uint_as_float((254u - eb) << 23);
                }
            }
            // store sweep: (second) pass over the accumulator, 16-bit pack, staged TMA stores
            if (nchunks > 0) {
                float l4[4] = {0.f, 0.f, 0.f, 0.f};
                const float ms = st_shift * kLog2e;
                if (!(p.debug & 16)) tc_ld32_issue(t_row, v[0]);
#pragma unroll
                for (int c = 0; c < kSub / 32; ++c) {
                    if (c < nchunks) {
                        if (!(p.debug & 16)) {
                            tc_ld_wait(v[c & 1]);
                            if (c + 1 < nchunks) tc_ld32_issue(t_row + (c + 1) * 32, v[(c + 1) & 1]);
                        }
                        float a[32];
#pragma unroll
                        for (int e = 0; e < 32; ++e) a[e] = __uint_as_float(v[c & 1][e]);
                        uint32_t w[16];
                        if (p.norm == KF_NORM_NONE) {
                            epilogue32(a, p, bias_t ? bias_t + c * 32 : nullptr, row, n0 + cb + c * 32, row_ok);
#pragma unroll
                            for (int e = 0; e < 16; ++e) w[e] = pack_bf16(a[2 * e], a[2 * e + 1]);
                        } else if (p.norm == KF_NORM_SOFTMAX) {
                            const bool full = (c + 1) * 32 <= ncols;
#pragma unroll
                            for (int e = 0; e < 32; ++e) {
                                a[e] = fast_ex2(fmaf(a[e], kLog2e, -ms));
                                if (full || c * 32 + e < ncols) l4[e & 3] += a[e];
                            }
#pragma unroll
                            for (int e = 0; e < 16; ++e) w[e] = pack_bf16(a[2 * e], a[2 * e + 1]);
                        } else {
#pragma unroll
                            for (int e = 0; e < 16; ++e) w[e] = pack_f16(a[2 * e] * mult, a[2 * e + 1] * mult);
                        }
                        if (row_ok && !(p.debug & 8)) store_row32(yrow + c * 32, w, ncols - c * 32);
                    }
                }
                if (p.norm == KF_NORM_SOFTMAX) st_s1 = (l4[0] + l4[1]) + (l4[2] + l4[3]);
            }
            if (p.debug & 256) {                            // timing experiment: a 5 us longer epilogue
                const long long t0 = clock64();
                while (clock64() - t0 < 10000) {}
            }
            // all TMEM accesses of this accumulator are done: hand it back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (CG == 2 && rank != 0) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));
                else mbar_arrive(tempty_bar(acc));
            }
            if (p.norm != KF_NORM_NONE && row_ok && nchunks > 0)
                p.partials[((size_t)mb * BM + q * 32 + lane) * p.nsub + (nb * 2 + half)] =
                    make_float4(st_shift, st_s1, st_s2, st_scale);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();                    // neither CTA leaves while the peer may still signal it
    if (warp == 1) {
        if (*abort_flag) {
            // give copies and MMAs in flight a bounded time to land before TMEM goes away
            for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        }
        tc_fence_after();
        if (CG == 2)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                         "r"((uint32_t)kTmemCols)
                         : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                         "r"((uint32_t)kTmemCols)
                         : "memory");
    }
}

// ------------------------------------------------------------------------------ finishing kernel
// WPR warps per row (1, 2, 4 or 8; a CTA of 8 warps holds 8 / WPR rows): merge the row's per-sub-tile
// partials (warp shuffles + one shared-memory hop across the row's warps), then rescale the 16-bit
// intermediates of the row in place with up to 8 independent 128-bit accesses in flight per lane.
constexpr int kFinWarps = 8;

template <bool IS_MAX>
__device__ __forceinline__ float fin_group_reduce(float v, int wpr, int warp, float* red) {
    v = IS_MAX ? warp_max(v) : warp_sum(v);
    if (wpr == 1) return v;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[warp] = v;
    __syncthreads();
    const int g0 = (warp / wpr) * wpr;
    float t = red[g0];
    for (int i = 1; i < wpr; ++i) t = IS_MAX ? fmaxf(t, red[g0 + i]) : t + red[g0 + i];
    return t;
}

__global__ void __launch_bounds__(kFinWarps * 32)
tc_rownorm_finish_kernel(__nv_bfloat16* Y, long long ldy, int M, int N, int nsub, int wpr,
                         const float4* __restrict__ partials, int norm, const __nv_bfloat16* __restrict__ gamma,
                         const __nv_bfloat16* __restrict__ beta, float eps) {
    extern __shared__ float2 coef_smem[];               // per row of the CTA: nsub x {multiplier, offset}
    __shared__ float red[kFinWarps];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rows_per_cta = kFinWarps / wpr;
    const int grow = warp / wpr;                         // row of this CTA
    const int gt = (warp % wpr) * 32 + lane, gsize = wpr * 32;     // thread index / count within the row's group
    long long row = (long long)blockIdx.x * rows_per_cta + grow;
    const bool live = row < M;
    if (!live) row = M - 1;                              // keep every thread in the barriers; stores are skipped
    float2* coef = coef_smem + (size_t)grow * nsub;
    const float4* pr = partials + (size_t)row * nsub;   // rows of a padded row block are contiguous
    float rstd = 1.f;

    if (norm == KF_NORM_SOFTMAX) {
        float m = -INFINITY;
        for (int s = gt; s < nsub; s += gsize) m = fmaxf(m, pr[s].x);
        m = fin_group_reduce<true>(m, wpr, warp, red);
        float l = 0.f;
        for (int s = gt; s < nsub; s += gsize) {
            const float4 q = pr[s];
            const float f = fast_ex2((q.x - m) * kLog2e);
            coef[s] = make_float2(f, 0.f);
            l = fmaf(q.y, f, l);
        }
        rstd = 1.0f / fin_group_reduce<false>(l, wpr, warp, red);
    } else if (norm == KF_NORM_LAYERNORM) {
        float sum = 0.f;
        for (int s = gt; s < nsub; s += gsize) {
            const float4 q = pr[s];
            const float cnt = (float)min(kSub, N - s * kSub);
            sum += q.x * cnt + q.y;               // sum of a over the sub-tile = shift * count + sum(a - shift)
        }
        const float mean = fin_group_reduce<false>(sum, wpr, warp, red) / (float)N;
        float m2 = 0.f;
        for (int s = gt; s < nsub; s += gsize) {
            const float4 q = pr[s];
            const float cnt = (float)min(kSub, N - s * kSub);
            const float dmean = q.y / cnt;                       // sub-tile mean minus its shift
            const float m2_t = fmaxf(q.z - q.y * dmean, 0.f);    // centred sum of squares of the sub-tile
            const float d = q.x + dmean - mean;
            m2 += fmaf(cnt * d, d, m2_t);                        // Chan's merge
            coef[s] = make_float2(q.w, q.x - mean);
        }
        rstd = rsqrtf(fin_group_reduce<false>(m2, wpr, warp, red) / (float)N + eps);
    } else {
        float ss = 0.f;
        for (int s = gt; s < nsub; s += gsize) {
            const float4 q = pr[s];
            ss += q.z;
            coef[s] = make_float2(q.w, 0.f);
        }
        rstd = rsqrtf(fin_group_reduce<false>(ss, wpr, warp, red) / (float)N + eps);
    }
    __syncthreads();                                     // coef of the row is complete
    if (!live) return;

    uint4* yr = reinterpret_cast<uint4*>(Y + row * ldy);
    const uint4* gv = reinterpret_cast<const uint4*>(gamma);
    const uint4* bv = reinterpret_cast<const uint4*>(beta);
    const int NV = N / 8;
    constexpr int U = 4;                                 // vectors in flight per lane
    for (int i0 = gt; i0 < NV; i0 += gsize * U) {
        uint4 raw[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int idx = i0 + u * gsize;
            if (idx < NV) raw[u] = yr[idx];
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int idx = i0 + u * gsize;
            if (idx >= NV) break;
            float f[8];
            const float2 c = coef[idx / (kSub / 8)];
            if (norm == KF_NORM_SOFTMAX) {
                unpack<__nv_bfloat16>(raw[u], f);
                const float k = c.x * rstd;
#pragma unroll
                for (int e = 0; e < 8; ++e) f[e] *= k;
            } else {
                unpack_f16x8(raw[u], f);
                float g[8], b[8];
                if (gamma) unpack<__nv_bfloat16>(__ldg(gv + idx), g);
                if (beta && norm == KF_NORM_LAYERNORM) unpack<__nv_bfloat16>(__ldg(bv + idx), b);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    float o = fmaf(f[e], c.x, c.y) * rstd;
                    if (gamma) o *= g[e];
                    if (beta && norm == KF_NORM_LAYERNORM) o += b[e];
                    f[e] = o;
                }
            }
            yr[idx] = pack<__nv_bfloat16>(f);
        }
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
              uint32_t box_rows, CUtensorMapSwizzle swizzle, CUtensorMapL2promotion promo) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, promo,
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
// Status block + per-row partial statistics for up to kStaticMaxTiles output tiles (8 MiB + 256 B).
// Every device that loads this library carries the array until the process exits.  In host code
// the name below is only a handle for cudaGetSymbolAddress; kernels receive the device address.
constexpr size_t kStaticMaxTiles = 2048;
constexpr size_t kStaticScratchBytes = kStatusBytes + kStaticMaxTiles * 2 * BM * sizeof(float4);
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

void tc_tile_shape(int cta_group, int* bm, int* bn, int* bk, int* stages, int* epi_warps) {
    *bm = BM * cta_group; *bn = BN; *bk = BK; *epi_warps = kEpiWarps;
    *stages = cta_group == 2 ? Cfg<2>::kStages : Cfg<1>::kStages;
}

// CTA pairs pay off as soon as there are two row blocks to pair up
int tc_default_cta_group(long long M, long long N) {
    (void)N;
    return M > BM ? 2 : 1;
}

size_t tc_partials_bytes(long long M, long long N) {
    const long long tm = (M + BM - 1) / BM, nsub = (N + kSub - 1) / kSub;
    return (size_t)tm * BM * nsub * sizeof(float4);
}

int tc_default_grid(long long M, long long N, int cta_group) {
    const long long tm = (M + BM - 1) / BM, tn = (N + BN - 1) / BN;
    const long long units = ((tm + cta_group - 1) / cta_group) * tn;
    const long long slots = sm_count() / cta_group;
    return (int)((units < slots ? units : slots) * cta_group);
}

kf_status launch_tc_linear(const void* X, long long ldx, const void* W, long long ldw, void* Y, long long ldy,
                           long long M, long long N, long long K, const EpilogueParams& ep, const RowNormParams& rn,
                           void* ws, int cta_group, int grid_override, cudaStream_t st, int* grid_out) {
    if (cta_group != 1 && cta_group != 2) return KF_ERR_INVALID_ARG;
    {   // opt in to the large dynamic shared memory once per device
        static std::mutex mu;
        static bool done[64] = {};
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return KF_ERR_CUDA;
        std::lock_guard<std::mutex> lock(mu);
        if (!done[dev]) {
            if (cudaFuncSetAttribute(tc_linear_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)kSmemAlloc) != cudaSuccess ||
                cudaFuncSetAttribute(tc_linear_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)kSmemAlloc) != cudaSuccess)
                return KF_ERR_CUDA;
            done[dev] = true;
        }
    }

    CUtensorMap tmX, tmW;
    if (!make_map(&tmX, X, M, K, ldx, BK, BM, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B) ||
        !make_map(&tmW, W, N, K, ldw, BK, BN / cta_group, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B))
        return KF_ERR_CUDA;

    TcParams p;
    p.M = (int)M; p.N = (int)N; p.K = (int)K;
    p.tiles_m = (int)((M + BM - 1) / BM);
    p.tiles_n = (int)((N + BN - 1) / BN);
    p.nsub = (int)((N + kSub - 1) / kSub);
    p.bias = static_cast<const __nv_bfloat16*>(ep.bias);
    p.residual = static_cast<const __nv_bfloat16*>(ep.residual);
    p.ldr = ep.ldr;
    p.act = ep.act;
    p.scale = ep.scale;
    p.norm = rn.norm;
    p.partials = reinterpret_cast<float4*>(static_cast<uint8_t*>(ws) + kStatusBytes);
    p.status = static_cast<uint32_t*>(ws);
    p.Y = static_cast<__nv_bfloat16*>(Y);
    p.ldy = ldy;
    static const int debug_mode = [] {
        const char* e = std::getenv("KF_TC_DEBUG");
        return e ? std::atoi(e) : 0;
    }();
    p.debug = debug_mode;
    static const long long timeout_cycles = [] {           // KF_TC_TIMEOUT_MS shortens the limit (tests)
        const char* e = std::getenv("KF_TC_TIMEOUT_MS");
        const long long ms = e ? std::atoll(e) : 0;
        return ms > 0 ? ms * 2000000ll : kTimeoutCycles;    // ~2 GHz clock64
    }();
    p.timeout_cycles = timeout_cycles;

    int grid = tc_default_grid(M, N, cta_group);
    if (grid_override > 0 && grid_override < grid) grid = grid_override - grid_override % cta_group;
    if (grid < cta_group) grid = cta_group;
    if (grid_out) *grid_out = grid;
    // finishing pass: one warp per row keeps the most rows in flight (measured best on C4 and C5);
    // more warps per row only for very long rows, whose coefficient table would not fit otherwise
    int wpr = 1;
    while (wpr < kFinWarps && (size_t)p.nsub * (kFinWarps / wpr) * sizeof(float2) > 40 * 1024) wpr <<= 1;
    static const int env_wpr = [] {
        const char* e = std::getenv("KF_FIN_WPR");
        return e ? std::atoi(e) : 0;
    }();
    if (env_wpr == 1 || env_wpr == 2 || env_wpr == 4 || env_wpr == 8) wpr = env_wpr;
    const int fin_rows = kFinWarps / wpr;
    const size_t fin_smem = (size_t)p.nsub * fin_rows * sizeof(float2);
    if (rn.norm != KF_NORM_NONE && fin_smem > 48 * 1024) return KF_ERR_UNSUPPORTED;   // N beyond ~780k
    if (cta_group == 2) {
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
        if (cudaLaunchKernelEx(&lc, tc_linear_kernel<2>, tmX, tmW, p) != cudaSuccess) {
            cudaGetLastError();
            return KF_ERR_CUDA;
        }
    } else {
        tc_linear_kernel<1><<<grid, kThreads, kSmemAlloc, st>>>(tmX, tmW, p);
    }
    if (cudaGetLastError() != cudaSuccess) return KF_ERR_CUDA;
    if (g_split_event && cudaEventRecord(g_split_event, st) != cudaSuccess) return KF_ERR_CUDA;

    if (rn.norm != KF_NORM_NONE) {
        tc_rownorm_finish_kernel<<<(unsigned)((M + fin_rows - 1) / fin_rows), kFinWarps * 32, fin_smem, st>>>(
            static_cast<__nv_bfloat16*>(Y), ldy, (int)M, (int)N, p.nsub, wpr, p.partials, rn.norm,
            static_cast<const __nv_bfloat16*>(rn.gamma), static_cast<const __nv_bfloat16*>(rn.beta), rn.eps);
        if (cudaGetLastError() != cudaSuccess) return KF_ERR_CUDA;
    }
    return KF_OK;
}

}  // namespace kf
