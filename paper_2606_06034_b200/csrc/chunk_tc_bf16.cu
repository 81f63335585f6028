// Tensor-core kernel (tcgen05 + TMEM + TMA) for the bf16 chunk-prepare path.
//
// Work item = one tile of 128 consecutive tokens of one (batch, value head): 128 / C chunks, which
// sit as diagonal blocks of every 128 x 128 operand (chunks are independent, so the tile's matrices
// are block diagonal). Thread t of the four compute warps owns row t of the tile (TMEM lane t); a
// fifth warp's lane 0 issues the TMA loads and every tcgen05.mma.
//
// Per tile (paper's notation, Abar = -A, Sec. 3 / Alg. 1):
//   G = K K^T                         tcgen05.mma, K tile staged by TMA (128B swizzle)      -> TMEM
//   Abar_ij = -beta_i e^{g_i-g_j} G_ij (i > j)                                  registers, fp32
//   L = T0 - I = band_{1<=i-j<=N}(sum_n Abar^n)  (Eq. 7, 10, 11), by the distance recursion
//       L_d[i] = Abar[i,i-d] + sum_{e<d} Abar[i,i-e] L_{d-e}[i-e], which equals the masked sum exactly
//   E = Abar + Abar L  on i-j > N, exactly 0 inside the band (Eq. 13)               registers, fp32
//   X_1 = E, X_{k+1} = E + X_k E  (S-1 dependent MMAs; X as bf16 A operand in TMEM, E as B in smem)
//   far = X_S + L X_S = T - I - L                                                     (one MMA)
//   T = I + L + far  -> Tinv
//   W = (I + L) diag(beta) K  [fp32 FMAs on the band]  +  (far diag(beta)) K  [MMA], same for U with V
// Only small quantities (E, X, far) pass through bf16 MMA operands; the identity and the O(1) band
// stay in fp32, which keeps the result within bf16 output rounding of the fp64 definition even for
// strongly correlated keys.
//
// The forward-substitution comparison (Eq. 2-3) replaces the L/E/X/far steps by a column-parallel
// substitution in shared memory and reuses everything else.
#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace gdn {
namespace {

using namespace sm100;

constexpr int kTile = 128;            // rows per work item
constexpr int kComputeThreads = 128;  // one per tile row
constexpr int kThreads = 160;         // + one control warp
constexpr int kD = 128;               // d_k = d_v
constexpr float kLog2e = 1.4426950408889634f;

// TMEM column map (256 columns allocated)
constexpr uint32_t kR0 = 0, kR1 = 64, kR2 = 128, kAS = 192, kTmemCols = 256;

struct Params {
    const float* beta;
    const float* g;
    __nv_bfloat16* W;
    __nv_bfloat16* U;
    __nv_bfloat16* Tinv;
    int* status;
    int H_k, H_v, T, group, n_tt;  // n_tt: tiles per head
    int N, S;
    long long n_tiles;
};

template <int C, int NB>
struct Smem {
    static constexpr int kK = 0;                        // 32 KB, two [128][64] bf16 sub-tiles, 128B swizzle
    static constexpr int kV = 32768;                    // 32 KB
    static constexpr int kEB = 65536;                   // B operand written by threads: 128 x C bf16
    static constexpr int kEBBytes = kTile * C * 2;
    static constexpr int kSH = kEB + kEBBytes;          // column form of the band: [128 + 8][NBP] floats
    static constexpr int NBP = (NB <= 3) ? 4 : 8;
    static constexpr int kSHBytes = (kTile + 8) * NBP * 4;
    static constexpr int kRB = kSH + kSHBytes;          // row form of the band: [128][NBP] floats
    static constexpr int kRBBytes = kTile * NBP * 4;
    static constexpr int kBeta = kRB + kRBBytes;        // 128 floats
    static constexpr int kG = kBeta + 512;              // 128 floats
    static constexpr int kFwd = kG + 512;               // forward substitution only: fp32 [128][C + 4]
    static constexpr int kTotalNeumann = kFwd;
    static constexpr int kTotalFwd = kFwd + kTile * (C + 4) * 4;
};

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void compute_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// bounded mbarrier wait: polls, and every 1024 polls compares the clock with a one-second budget
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity) {
    const long long t0 = clock64();
    uint32_t i = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++i & 1023u) == 0 && clock64() - t0 > 2000000000LL) return false;
    }
    return true;
}


// Writes this row's packed bf16 diagonal block (C / 2 32-bit columns) into the A-operand slot.
// tcgen05.st takes one address per warp: for C = 16 a warp holds two chunks, so the warp stores a
// 16-column window in which each half-warp fills its own half and zero-fills the other.
template <int C>
__device__ __forceinline__ void store_a_operand(uint32_t lane_base, int t, const uint32_t (&pk)[C / 2]) {
    constexpr int PC = C / 2;
    if constexpr (PC >= 16) {
        const int cb = t - (t % C);
#pragma unroll
        for (int c = 0; c < PC / 16; ++c) {
            uint32_t r16[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) r16[i] = pk[c * 16 + i];
            tmem_st16(lane_base + kAS + cb / 2 + c * 16, r16);
        }
    } else {
        const int wb = t & ~31;
        const bool upper = (t & 16) != 0;
        uint32_t r16[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            r16[i] = upper ? 0u : pk[i];
            r16[8 + i] = upper ? pk[i] : 0u;
        }
        tmem_st16(lane_base + kAS + wb / 2, r16);
    }
}

// Reads this row's C columns of a block-diagonal 128-column accumulator (the Gram matrix).
template <int C>
__device__ __forceinline__ void load_diag_block(uint32_t lane_base, uint32_t col0, int t, float (&a)[C]) {
    if constexpr (C >= 32) {
        const int cb = t - (t % C);
#pragma unroll
        for (int c0 = 0; c0 < C; c0 += 32) {
            uint32_t r[32];
            tmem_ld32(lane_base + col0 + cb + c0, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) a[c0 + i] = __uint_as_float(r[i]);
        }
    } else {
        const int wb = t & ~31;
        const bool upper = (t & 16) != 0;
        uint32_t r[32];
        tmem_ld32(lane_base + col0 + wb, r);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 16; ++i) a[i] = __uint_as_float(upper ? r[16 + i] : r[i]);
    }
}

// Reads C consecutive accumulator columns starting at col0 (same address for the whole warp).
template <int C>
__device__ __forceinline__ void load_cols(uint32_t lane_base, uint32_t col0, uint32_t (&r)[C]) {
    if constexpr (C >= 32) {
#pragma unroll
        for (int c0 = 0; c0 < C; c0 += 32) {
            uint32_t q[32];
            tmem_ld32(lane_base + col0 + c0, q);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[c0 + i] = q[i];
        }
    } else {
        uint32_t q[16];
        tmem_ld16(lane_base + col0, q);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 16; ++i) r[i] = q[i];
    }
}

template <int C, int NB, int MODE>
__global__ void __launch_bounds__(kThreads, 2)
chunk_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const Params p) {
    using L = Smem<C, NB>;
    constexpr int NBP = L::NBP;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sK = smem + L::kK;
    uint8_t* sV = smem + L::kV;
    uint8_t* sEB = smem + L::kEB;
    float* sSH = reinterpret_cast<float*>(smem + L::kSH);
    float* sRB = reinterpret_cast<float*>(smem + L::kRB);
    float* sbeta = reinterpret_cast<float*>(smem + L::kBeta);
    float* sg = reinterpret_cast<float*>(smem + L::kG);

    __shared__ uint64_t bar_k, bar_v, bar_mma, bar_opnd, bar_free;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;

    if (tid == 0) {
        mbar_init(&bar_k, 1);
        mbar_init(&bar_v, 1);
        mbar_init(&bar_mma, 1);
        mbar_init(&bar_opnd, kComputeThreads);
        mbar_init(&bar_free, kComputeThreads);
        abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 4) {
        tmem_alloc(&tmem_base_s, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_s;

    const int N = p.N, S = p.S;
    // width of the band kept in fp32 registers (lb[]): the order N, or all of NB for forward substitution
    const int n_band = (MODE == INV_NEUMANN) ? N : NB;
    // number of MMA rounds between the A-build and the W/U products
    const int n_rounds = (MODE == INV_NEUMANN) ? (S >= 1 ? S : 0) : 0;

    if (warp == 4) {
        // ------------------------------------------------------------------ control warp
        if ((tid & 31) == 0) {
            tma_prefetch_desc(&tmK);
            tma_prefetch_desc(&tmV);
            uint32_t par_kv = 0, par_opnd = 0, par_free = 0;
            bool ok = true;
            bool first = true;
            const uint32_t idesc_g = instr_desc(128, 128, 1, 1, 0, 0, 1);
            const uint32_t idesc_c = instr_desc(128, C, 1, 1, 0, 1, 1);
            const uint32_t idesc_w = instr_desc(128, 64, 1, 1, 0, 1, 1);
            const uint32_t sK_a = smem_u32(sK), sV_a = smem_u32(sV), sEB_a = smem_u32(sEB);
            for (long long tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x) {
                const int gi = static_cast<int>(tile % p.group);
                const long long y = tile / p.group;
                const int tt = static_cast<int>(y % p.n_tt);
                const long long bhk = y / p.n_tt;
                const long long b = bhk / p.H_k;
                const int hk = static_cast<int>(bhk % p.H_k);
                const long long bhv = b * p.H_v + (long long)hk * p.group + gi;
                const int t0 = tt * kTile;
                if (!first) {
                    if (!wait_bar(&bar_free, par_free)) { ok = false; break; }
                    par_free ^= 1;
                }
                first = false;
                mbar_arrive_expect_tx(&bar_k, 32768);
                tma_load_3d(sK, &tmK, &bar_k, 0, t0, static_cast<int>(bhk));
                tma_load_3d(sK + 16384, &tmK, &bar_k, 64, t0, static_cast<int>(bhk));
                mbar_arrive_expect_tx(&bar_v, 32768);
                tma_load_3d(sV, &tmV, &bar_v, 0, t0, static_cast<int>(bhv));
                tma_load_3d(sV + 16384, &tmV, &bar_v, 64, t0, static_cast<int>(bhv));
                if (!wait_bar(&bar_k, par_kv)) { ok = false; break; }
                tc_fence_after_sync();
                // G = K K^T into R0..R1 (128 columns)
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t d = smem_desc(sK_a + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024, SWZ_128B);
                    mma_f16_ss(tmem + kR0, d, d, idesc_g, ks > 0);
                }
                mma_commit(&bar_mma);
                for (int r = 0; r < n_rounds && ok; ++r) {
                    if (!wait_bar(&bar_opnd, par_opnd)) { ok = false; break; }
                    par_opnd ^= 1;
                    tc_fence_after_sync();
                    const uint32_t dcol = (r < n_rounds - 1) ? kR2 : kR0;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint64_t bd = smem_desc(sEB_a + ks * 256, 128, 2048, SWZ_NONE);
                        mma_f16_ts(tmem + dcol, tmem + kAS + ks * 8, bd, idesc_c, ks > 0);
                    }
                    mma_commit(&bar_mma);
                }
                if (!ok) break;
                // W and U: A = far * diag(beta) in TMEM, B = the K / V tile as an MN-major operand
                if (!wait_bar(&bar_opnd, par_opnd)) { ok = false; break; }
                par_opnd ^= 1;
                if (!wait_bar(&bar_v, par_kv)) { ok = false; break; }
                par_kv ^= 1;
                tc_fence_after_sync();
#pragma unroll
                for (int part = 0; part < 3; ++part) {
                    const uint32_t base = (part < 2) ? (sK_a + part * 16384) : sV_a;
                    const uint32_t dcol = (part == 0) ? kR0 : (part == 1 ? kR1 : kR2);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint64_t bd = smem_desc(base + ks * 2048, 16384, 1024, SWZ_128B);
                        mma_f16_ts(tmem + dcol, tmem + kAS + ks * 8, bd, idesc_w, ks > 0);
                    }
                }
                mma_commit(&bar_mma);
                if (!wait_bar(&bar_opnd, par_opnd)) { ok = false; break; }  // R0 read out
                par_opnd ^= 1;
                tc_fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t bd = smem_desc(sV_a + 16384 + ks * 2048, 16384, 1024, SWZ_128B);
                    mma_f16_ts(tmem + kR0, tmem + kAS + ks * 8, bd, idesc_w, ks > 0);
                }
                mma_commit(&bar_mma);
            }
            if (!ok) {
                atomicExch(p.status, GDN_ERR_TIMEOUT);
                atomicExch(&abort_flag, 1);
            }
        }
    } else {
        // ------------------------------------------------------------------ compute warps
        const int t = tid;                 // tile row
        const int il = t % C;              // row inside its chunk
        const int cb = t - il;             // first tile row of the chunk
        const uint32_t lane_base = tmem + (static_cast<uint32_t>(warp * 32) << 16);
        uint32_t par_mma = 0, par_kv = 0;
        bool ok = true;

        {  // the A-operand slot keeps zeros outside the diagonal blocks for the whole kernel
            uint32_t z[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) z[i] = 0u;
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_st16(lane_base + kAS + c * 16, z);
            tmem_wait_st();
        }

        for (long long tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x) {
            const int gi = static_cast<int>(tile % p.group);
            const long long y = tile / p.group;
            const int tt = static_cast<int>(y % p.n_tt);
            const long long bhk = y / p.n_tt;
            const long long b = bhk / p.H_k;
            const int hk = static_cast<int>(bhk % p.H_k);
            const long long bhv = b * p.H_v + (long long)hk * p.group + gi;
            const int t0 = tt * kTile;
            const bool row_valid = (t0 + t) < p.T;
            const long long grow = bhv * (long long)p.T + t0 + t;  // global token row (value-head space)

            float bi = 0.f, gi_ = 0.f;
            if (row_valid) {
                bi = __ldg(p.beta + grow);
                gi_ = __ldg(p.g + grow);
            }
            compute_barrier();  // everyone is done with the previous tile's shared arrays
            sbeta[t] = bi;
            sg[t] = gi_;
#pragma unroll
            for (int e = 0; e < NBP; ++e) sSH[t * NBP + e] = 0.f;
            if (t < 8) {
#pragma unroll
                for (int e = 0; e < NBP; ++e) sSH[(kTile + t) * NBP + e] = 0.f;
            }
            compute_barrier();

            // ---- A-build: row of Abar from the Gram block in TMEM
            if (!wait_bar(&bar_mma, par_mma)) { ok = false; break; }
            par_mma ^= 1;
            tc_fence_after_sync();
            float a[C];
            load_diag_block<C>(lane_base, kR0, t, a);
            float ab[NB + 1];  // ab[e] = Abar[i][i-e]
#pragma unroll
            for (int e = 0; e <= NB; ++e) ab[e] = 0.f;
            {
                const float gs = gi_ * kLog2e;
                const float4* sg4 = reinterpret_cast<const float4*>(sg + cb);
#pragma unroll
                for (int j4 = 0; j4 < C / 4; ++j4) {
                    const float4 gq = sg4[j4];
                    const float gj[4] = {gq.x, gq.y, gq.z, gq.w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int j = j4 * 4 + q;
                        float v = 0.f;
                        if (j < il) v = -bi * fast_exp2(fmaf(-gj[q], kLog2e, gs)) * a[j];
                        a[j] = v;
#pragma unroll
                        for (int e = 1; e <= NB; ++e)
                            if (j == il - e) ab[e] = v;
                    }
                }
            }

            float lb[NB + 1];  // lb[d] = L[i][i-d], the band of T0 - I
#pragma unroll
            for (int e = 0; e <= NB; ++e) lb[e] = 0.f;

            if constexpr (MODE == INV_NEUMANN) {
                // ---- band of the masked Neumann sum by distance recursion
                lb[1] = ab[1];
                sRB[t * NBP + 0] = lb[1];
#pragma unroll
                for (int d = 2; d <= NB; ++d) {
                    compute_barrier();
                    float v = ab[d];
#pragma unroll
                    for (int e = 1; e < d; ++e) {
                        const int r = (t - e) > 0 ? (t - e) : 0;
                        v = fmaf(ab[e], sRB[r * NBP + (d - e - 1)], v);
                    }
                    lb[d] = (d <= N) ? v : 0.f;
                    if (d < NB) sRB[t * NBP + (d - 1)] = lb[d];
                }
                if (N < 1) lb[1] = 0.f;
                // column form: SH[j][e-1] = L[j+e][j]
#pragma unroll
                for (int e = 1; e <= NB; ++e)
                    if (il - e >= 0) sSH[(t - e) * NBP + (e - 1)] = lb[e];
                compute_barrier();

                // ---- E = Abar + Abar L on i-j > N (in place over a[])
#pragma unroll
                for (int j = 0; j < C; ++j) {
                    float v = 0.f;
                    if (il - j > N) {
                        v = a[j];
                        if constexpr (NBP == 4) {
                            const float4 c4 = *reinterpret_cast<const float4*>(sSH + (cb + j) * 4);
                            if (j + 1 < C) v = fmaf(a[(j + 1 < C) ? j + 1 : j], c4.x, v);
                            if (j + 2 < C) v = fmaf(a[(j + 2 < C) ? j + 2 : j], c4.y, v);
                            if (j + 3 < C) v = fmaf(a[(j + 3 < C) ? j + 3 : j], c4.z, v);
                        } else {
                            const float4 c4 = *reinterpret_cast<const float4*>(sSH + (cb + j) * 8);
                            const float4 d4 = *reinterpret_cast<const float4*>(sSH + (cb + j) * 8 + 4);
                            const float cc[7] = {c4.x, c4.y, c4.z, c4.w, d4.x, d4.y, d4.z};
#pragma unroll
                            for (int e = 1; e <= NB; ++e)
                                if (j + e < C) v = fmaf(a[(j + e < C) ? j + e : j], cc[e - 1], v);
                        }
                    }
                    a[j] = v;
                }
                // now a[] = E row. Chain: x = X_k row.
                float x[C];
#pragma unroll
                for (int j = 0; j < C; ++j) x[j] = (S >= 1) ? a[j] : 0.f;

                if (S >= 1) {
                    // E as B operand (MN-major, no swizzle): 16-byte chunk c of row t at c * 2048 + t * 16
#pragma unroll
                    for (int c = 0; c < C / 8; ++c) {
                        uint4 v;
                        v.x = pack_bf16x2(a[c * 8 + 0], a[c * 8 + 1]);
                        v.y = pack_bf16x2(a[c * 8 + 2], a[c * 8 + 3]);
                        v.z = pack_bf16x2(a[c * 8 + 4], a[c * 8 + 5]);
                        v.w = pack_bf16x2(a[c * 8 + 6], a[c * 8 + 7]);
                        *reinterpret_cast<uint4*>(sEB + c * 2048 + t * 16) = v;
                    }
                }
                for (int k = 1; k <= S; ++k) {
                    // operand for round k: X_k (k < S) or the band L (k == S, "far" product with B = X_S)
                    if (k == S) {
#pragma unroll
                        for (int c = 0; c < C / 8; ++c) {
                            uint4 v;
                            v.x = pack_bf16x2(x[c * 8 + 0], x[c * 8 + 1]);
                            v.y = pack_bf16x2(x[c * 8 + 2], x[c * 8 + 3]);
                            v.z = pack_bf16x2(x[c * 8 + 4], x[c * 8 + 5]);
                            v.w = pack_bf16x2(x[c * 8 + 6], x[c * 8 + 7]);
                            *reinterpret_cast<uint4*>(sEB + c * 2048 + t * 16) = v;
                        }
                    }
                    {
                        constexpr int PC = C / 2;  // packed columns of this row's diagonal block
                        uint32_t pk[PC];
#pragma unroll
                        for (int jp = 0; jp < PC; ++jp) {
                            float lo, hi;
                            if (k < S) {
                                lo = x[2 * jp];
                                hi = x[2 * jp + 1];
                            } else {
                                lo = 0.f;
                                hi = 0.f;
#pragma unroll
                                for (int e = 1; e <= NB; ++e) {
                                    if (2 * jp == il - e) lo = lb[e];
                                    if (2 * jp + 1 == il - e) hi = lb[e];
                                }
                            }
                            pk[jp] = pack_bf16x2(lo, hi);
                        }
                        store_a_operand<C>(lane_base, t, pk);
                    }
                    fence_proxy_async_smem();
                    tmem_wait_st();
                    tc_fence_before_sync();
                    mbar_arrive(&bar_opnd);
                    if (!wait_bar(&bar_mma, par_mma)) { ok = false; break; }
                    par_mma ^= 1;
                    tc_fence_after_sync();
                    const uint32_t dcol = (k < S) ? kR2 : kR0;
                    uint32_t dres[C];
                    load_cols<C>(lane_base, dcol, dres);
#pragma unroll
                    for (int i = 0; i < C; ++i) x[i] = ((k < S) ? a[i] : x[i]) + __uint_as_float(dres[i]);
                }
                if (!ok) break;
                // x[] = far row. Move into a[] for the common tail.
#pragma unroll
                for (int j = 0; j < C; ++j) a[j] = x[j];
            } else {
                // ---- forward substitution (Eq. 2-3), thread = column of its chunk
                float* sF = reinterpret_cast<float*>(smem + L::kFwd);
                constexpr int LDF = C + 4;
#pragma unroll
                for (int j = 0; j < C; ++j) sF[t * LDF + j] = a[j];
                compute_barrier();
                float xcol[C];  // xcol[k] = T[k][il] of this thread's chunk (column il)
#pragma unroll
                for (int i = 0; i < C; ++i) {
                    float acc = 0.f;
#pragma unroll
                    for (int k = 0; k < i; ++k) acc = fmaf(sF[(cb + i) * LDF + k], xcol[k], acc);
                    xcol[i] = (i > il) ? acc : ((i == il) ? 1.f : 0.f);
                }
                compute_barrier();  // everyone has read Abar
#pragma unroll
                for (int i = 0; i < C; ++i) sF[(cb + i) * LDF + il] = xcol[i];
                compute_barrier();
                // back to rows: a[] = far part, lb[] = band part
#pragma unroll
                for (int j = 0; j < C; ++j) {
                    const float v = sF[t * LDF + j];
                    const int dist = il - j;
                    a[j] = (dist > NB) ? v : 0.f;
#pragma unroll
                    for (int e = 1; e <= NB; ++e)
                        if (dist == e) lb[e] = v;
                }
            }

            // ---- T row -> Tinv
            if (p.Tinv != nullptr && row_valid) {
                __nv_bfloat16* trow = p.Tinv + (grow / C) * (long long)(C * C) + (long long)il * C;
#pragma unroll
                for (int c = 0; c < C / 8; ++c) {
                    float v[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const int j = c * 8 + q;
                        float val = a[j];
                        if (j == il) val = 1.f;
#pragma unroll
                        for (int e = 1; e <= NB; ++e)
                            if (j == il - e && e <= n_band) val = lb[e];
                        v[q] = val;
                    }
                    uint4 o;
                    o.x = pack_bf16x2(v[0], v[1]);
                    o.y = pack_bf16x2(v[2], v[3]);
                    o.z = pack_bf16x2(v[4], v[5]);
                    o.w = pack_bf16x2(v[6], v[7]);
                    *reinterpret_cast<uint4*>(trow + c * 8) = o;
                }
            }

            // ---- A operand for W/U: far * diag(beta)
            {
                constexpr int PC = C / 2;
                uint32_t pk[PC];
                const float2* sb2 = reinterpret_cast<const float2*>(sbeta + cb);
#pragma unroll
                for (int jp = 0; jp < PC; ++jp) {
                    const float2 bb = sb2[jp];
                    pk[jp] = pack_bf16x2(a[2 * jp] * bb.x, a[2 * jp + 1] * bb.y);
                }
                store_a_operand<C>(lane_base, t, pk);
                tmem_wait_st();
                tc_fence_before_sync();
                mbar_arrive(&bar_opnd);
            }

            // ---- W, U: band part on the FMA pipes, far part from the MMA
            float coef[NB + 1];
            coef[0] = bi;
#pragma unroll
            for (int e = 1; e <= NB; ++e) coef[e] = (il - e >= 0) ? lb[e] * sbeta[(t - e) > 0 ? (t - e) : 0] : 0.f;

            // the TMA barriers completed long ago; waiting on them here makes the tiles visible to this thread
            if (!wait_bar(&bar_k, par_kv) || !wait_bar(&bar_v, par_kv)) { ok = false; break; }
            par_kv ^= 1;
#pragma unroll 1
            for (int part = 0; part < 4; ++part) {
                // part 0: W[:, 0:64] (R0), 1: W[:, 64:128] (R1), 2: U[:, 0:64] (R2), 3: U[:, 64:128] (R0, second commit)
                const uint8_t* src = ((part < 2) ? sK : sV) + (part & 1) * 16384;
                float acc[64];
#pragma unroll
                for (int i = 0; i < 64; ++i) acc[i] = 0.f;
#pragma unroll
                for (int e = 0; e <= NB; ++e) {
                    const int r = (t - e) > 0 ? (t - e) : 0;
                    const float cf = coef[e];
                    const uint8_t* rowp = src + r * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint4 q = *reinterpret_cast<const uint4*>(rowp + ((c ^ (r & 7)) << 4));
                        acc[c * 8 + 0] = fmaf(cf, bf16_lo(q.x), acc[c * 8 + 0]);
                        acc[c * 8 + 1] = fmaf(cf, bf16_hi(q.x), acc[c * 8 + 1]);
                        acc[c * 8 + 2] = fmaf(cf, bf16_lo(q.y), acc[c * 8 + 2]);
                        acc[c * 8 + 3] = fmaf(cf, bf16_hi(q.y), acc[c * 8 + 3]);
                        acc[c * 8 + 4] = fmaf(cf, bf16_lo(q.z), acc[c * 8 + 4]);
                        acc[c * 8 + 5] = fmaf(cf, bf16_hi(q.z), acc[c * 8 + 5]);
                        acc[c * 8 + 6] = fmaf(cf, bf16_lo(q.w), acc[c * 8 + 6]);
                        acc[c * 8 + 7] = fmaf(cf, bf16_hi(q.w), acc[c * 8 + 7]);
                    }
                }
                if (part == 0 || part == 3) {
                    if (!wait_bar(&bar_mma, par_mma)) { ok = false; break; }
                    par_mma ^= 1;
                    tc_fence_after_sync();
                }
                const uint32_t dcol = (part == 1) ? kR1 : (part == 2 ? kR2 : kR0);
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld32(lane_base + dcol + c0, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) acc[c0 + i] += __uint_as_float(r[i]);
                }
                if (part == 0) {  // R0 is free for the second half of U
                    tc_fence_before_sync();
                    mbar_arrive(&bar_opnd);
                }
                if (row_valid) {
                    __nv_bfloat16* dst = ((part < 2) ? p.W : p.U) + grow * kD + (part & 1) * 64;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        uint4 o;
                        o.x = pack_bf16x2(acc[c * 8 + 0], acc[c * 8 + 1]);
                        o.y = pack_bf16x2(acc[c * 8 + 2], acc[c * 8 + 3]);
                        o.z = pack_bf16x2(acc[c * 8 + 4], acc[c * 8 + 5]);
                        o.w = pack_bf16x2(acc[c * 8 + 6], acc[c * 8 + 7]);
                        *reinterpret_cast<uint4*>(dst + c * 8) = o;
                    }
                }
            }
            if (!ok) break;
            tc_fence_before_sync();
            mbar_arrive(&bar_free);
        }
        if (!ok) {
            atomicExch(p.status, GDN_ERR_TIMEOUT);
            atomicExch(&abort_flag, 1);
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 4) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, kTmemCols);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// [heads][T][128] bf16 tensor, boxes of 128 rows x 64 columns, 128-byte swizzle
bool make_tile_map(CUtensorMap* tm, const void* base, long long heads, int T) {
    EncodeTiledFn enc = get_encode_fn();
    if (enc == nullptr) return false;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(kD), static_cast<cuuint64_t>(T), static_cast<cuuint64_t>(heads)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(kD) * 2, static_cast<cuuint64_t>(T) * kD * 2};
    cuuint32_t box[3] = {64, 128, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int C, int NB, int MODE>
int launch_one(const CUtensorMap& tmK, const CUtensorMap& tmV, const Params& prm, cudaStream_t stream) {
    using L = Smem<C, NB>;
    const int smem = ((MODE == INV_NEUMANN) ? L::kTotalNeumann : L::kTotalFwd) + 1024;
    auto kern = chunk_tc_kernel<C, NB, MODE>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return GDN_ERR_LAUNCH;
    long long grid = prm.n_tiles < 2 * 148 ? prm.n_tiles : 2 * 148;
    kern<<<static_cast<int>(grid), kThreads, smem, stream>>>(tmK, tmV, prm);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_LAUNCH;
}

template <int C, int MODE>
int launch_c(const CUtensorMap& tmK, const CUtensorMap& tmV, const Params& prm, cudaStream_t stream) {
    if (MODE != INV_NEUMANN || prm.N <= 3) return launch_one<C, 3, MODE>(tmK, tmV, prm, stream);
    return launch_one<C, 7, MODE>(tmK, tmV, prm, stream);
}

}  // namespace

int launch_tc_bf16(const Problem& p, InverseMode mode, cudaStream_t stream) {
    if (p.d_k != kD || p.d_v != kD) return GDN_ERR_UNSUPPORTED;
    if (!(p.C == 16 || p.C == 32 || p.C == 64)) return GDN_ERR_UNSUPPORTED;
    if (mode == INV_NEUMANN && (p.order < 1 || p.order > 7)) return GDN_ERR_UNSUPPORTED;
    if (mode == INV_FWDSUBST_BLOCKED) return GDN_ERR_UNSUPPORTED;
    if ((long long)p.B * p.H_v * p.T == 0) return GDN_OK;
    int* status = device_status_word();
    if (status == nullptr) return GDN_ERR_LAUNCH;
    CUtensorMap tmK, tmV;
    if (!make_tile_map(&tmK, p.K, (long long)p.B * p.H_k, p.T)) return GDN_ERR_LAUNCH;
    if (!make_tile_map(&tmV, p.V, (long long)p.B * p.H_v, p.T)) return GDN_ERR_LAUNCH;
    Params prm;
    prm.beta = p.beta;
    prm.g = p.g;
    prm.W = static_cast<__nv_bfloat16*>(p.W);
    prm.U = static_cast<__nv_bfloat16*>(p.U);
    prm.Tinv = static_cast<__nv_bfloat16*>(p.Tinv);
    prm.status = status;
    prm.H_k = p.H_k;
    prm.H_v = p.H_v;
    prm.T = p.T;
    prm.group = p.H_v / p.H_k;
    prm.n_tt = (p.T + kTile - 1) / kTile;
    prm.N = p.order;
    prm.S = p.steps;
    prm.n_tiles = (long long)p.B * p.H_v * prm.n_tt;
    if (mode == INV_NEUMANN) {
        switch (p.C) {
            case 16: return launch_c<16, INV_NEUMANN>(tmK, tmV, prm, stream);
            case 32: return launch_c<32, INV_NEUMANN>(tmK, tmV, prm, stream);
            default: return launch_c<64, INV_NEUMANN>(tmK, tmV, prm, stream);
        }
    }
    switch (p.C) {
        case 16: return launch_c<16, INV_FWDSUBST_ROWS>(tmK, tmV, prm, stream);
        case 32: return launch_c<32, INV_FWDSUBST_ROWS>(tmK, tmV, prm, stream);
        default: return launch_c<64, INV_FWDSUBST_ROWS>(tmK, tmV, prm, stream);
    }
}

}  // namespace gdn
