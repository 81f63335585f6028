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
constexpr int kThreads = 128;
constexpr int kD = 128;               // d_k = d_v
constexpr float kLog2e = 1.4426950408889634f;

// TMEM column map (256 columns allocated):
//   R0..R1 (128 columns)  Gram matrix, later the W and then the U accumulator
//   R2     (64 columns)   accumulator of the residual rounds, later the low-half A operand of W/U
//   AS     (64 columns)   bf16 A operand (block diagonal, 128 x 128) of the residual rounds and of W/U
constexpr uint32_t kR0 = 0, kR2 = 128, kAS = 192, kTmemCols = 256;

#ifdef GDN_TRACE
__device__ long long g_trace[4096];
#define STAMP(slot) do { if (blockIdx.x == 0 && tid == 32 && trace_n < 100) { g_trace[trace_n * 2] = (slot); g_trace[trace_n * 2 + 1] = clock64(); ++trace_n; } } while (0)
#else
#define STAMP(slot) do { } while (0)
#endif

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
    // scratch: [EB | BR]. EB = E as the B operand of the residual rounds (128 x C bf16, core-matrix
    // layout); BR = one private packed-bf16 row per thread. Before EB/BR are in use the whole region
    // holds one private fp32 row per thread (Abar row, or the forward-substitution matrix).
    static constexpr int kEB = 65536;
    static constexpr int kEBBytes = kTile * C * 2;
    static constexpr int kBR = kEB + kEBBytes;
    static constexpr int kBRBytes = kTile * C * 2;
    static constexpr int NBP = (NB <= 3) ? 4 : 8;
    static constexpr int kScratchBytes = 32768;         // >= kEBBytes + kBRBytes; also the 4 x 8 KB store staging slices
    static constexpr int kSH = kEB + kScratchBytes;     // column form of the band: [128 + 8][NBP] floats
    static constexpr int kSHBytes = (kTile + 8) * NBP * 4;
    static constexpr int kRB = kSH + kSHBytes;          // row form of the band: [128][NBP] floats
    static constexpr int kRBBytes = kTile * NBP * 4;
    static constexpr int kBeta = kRB + kRBBytes;        // 128 floats
    static constexpr int kG = kBeta + 512;              // 128 floats
    static constexpr int kTotal = kG + 512;
};

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void compute_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// bounded mbarrier wait: polls, and every 1024 polls compares the clock with a budget of about a second
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t i = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++i & 1023u) == 0 && clock64() - t0 > 2000000000LL) return false;
    }
    return true;
}

// ---- private shared-memory rows (each thread touches only its own row; inline asm keeps the order)
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void sts16(uint32_t addr, uint16_t v) {
    asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr), "h"(v) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ float lds32f(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
// 16-byte chunk index after the bank swizzle, for rows of CPR chunks
template <int CPR>
__device__ __forceinline__ int swz(int t, int c) {
    if constexpr (CPR >= 8) return c ^ (t & 7);
    else if constexpr (CPR == 4) return c ^ ((t >> 1) & 3);
    else if constexpr (CPR == 2) return c ^ ((t >> 2) & 1);
    else return c;
}

// Builds a packed bf16 row of C entries that is zero except vals[e] at column il - e (e = 0..n_valid,
// skipped where il - e < 0), through the thread's private row in shared memory: registers cannot be
// indexed by a per-thread position, shared memory can.
template <int C, int NB>
__device__ __forceinline__ void build_band_row(uint32_t row_addr, int t, int il, int n_valid, const uint16_t (&vals)[NB + 1],
                                               uint32_t (&out)[C / 2]) {
    constexpr int CPR = C / 8;
#pragma unroll
    for (int c = 0; c < CPR; ++c) sts128(row_addr + (swz<CPR>(t, c) << 4), 0u, 0u, 0u, 0u);
#pragma unroll
    for (int e = 0; e <= NB; ++e) {
        const int j = il - e;
        if (j >= 0 && e <= n_valid) sts16(row_addr + (swz<CPR>(t, j >> 3) << 4) + (j & 7) * 2, vals[e]);
    }
#pragma unroll
    for (int c = 0; c < CPR; ++c) {
        const uint4 v = lds128(row_addr + (swz<CPR>(t, c) << 4));
        out[c * 4 + 0] = v.x;
        out[c * 4 + 1] = v.y;
        out[c * 4 + 2] = v.z;
        out[c * 4 + 3] = v.w;
    }
}

__device__ __forceinline__ uint16_t bf16_bits(float x) { return __bfloat16_as_ushort(__float2bfloat16_rn(x)); }
__device__ __forceinline__ float bf16_bits_to_f32(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }

// Writes this row's packed bf16 diagonal block (C / 2 32-bit columns) into a 64-column A-operand slot.
// tcgen05.st takes one address per warp: for C = 16 a warp holds two chunks, so the warp stores a
// 16-column window in which each half-warp fills its own half and zero-fills the other.
// FULL: also zero-fill the rest of the 64-column row (slot that held other data before).
template <int C, bool FULL>
__device__ __forceinline__ void store_a_operand(uint32_t slot_addr, int t, const uint32_t (&pk)[C / 2]) {
    constexpr int PC = C / 2;
    const int wb = (C >= 32) ? (t - (t % C)) : (t & ~31);  // first tile row of the warp-uniform window
    constexpr int WC = (PC >= 16) ? PC : 16;               // window width in columns
    const bool upper = (C < 32) && ((t & 16) != 0);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        // 16-column group c of the 64-column slot
        uint32_t r16[16];
        const int rel = c * 16 - wb / 2;  // position of this group relative to the window
        const bool inside = (rel >= 0) && (rel < WC);
        if (!FULL && !inside) continue;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            uint32_t v = 0u;
            if constexpr (PC >= 16) {
                // rel is 0 or 16 (C = 64) or 0 (C = 32) when inside
                if (inside) v = (PC == 32) ? ((rel == 0) ? pk[i] : pk[(16 + i) % PC]) : pk[i % PC];
            } else {
                if (inside) v = upper ? ((i >= 8) ? pk[i - 8] : 0u) : ((i < 8) ? pk[i] : 0u);
            }
            r16[i] = v;
        }
        tmem_st16(slot_addr + c * 16, r16);
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
__device__ __forceinline__ void load_cols(uint32_t lane_base, uint32_t col0, float (&r)[C]) {
    if constexpr (C >= 32) {
#pragma unroll
        for (int c0 = 0; c0 < C; c0 += 32) {
            uint32_t q[32];
            tmem_ld32(lane_base + col0 + c0, q);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[c0 + i] = __uint_as_float(q[i]);
        }
    } else {
        uint32_t q[16];
        tmem_ld16(lane_base + col0, q);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 16; ++i) r[i] = __uint_as_float(q[i]);
    }
}

struct TileCoord {
    int bhk, bhv;
    int t0;
};
// tile index -> (key head row, value head row, first token); tiles that share a key tile are adjacent.
// All counts fit 32 bits (checked by the launcher).
__device__ __forceinline__ TileCoord decode_tile(uint32_t tile, const Params& p) {
    TileCoord c;
    const uint32_t y = tile / static_cast<uint32_t>(p.group);
    const uint32_t gi = tile - y * p.group;
    const uint32_t bhk = y / static_cast<uint32_t>(p.n_tt);
    const uint32_t tt = y - bhk * p.n_tt;
    const uint32_t b = bhk / static_cast<uint32_t>(p.H_k);
    const uint32_t hk = bhk - b * p.H_k;
    c.bhk = static_cast<int>(bhk);
    c.bhv = static_cast<int>(b * p.H_v + hk * p.group + gi);
    c.t0 = static_cast<int>(tt) * kTile;
    return c;
}

template <int C, int NB, int MODE>
__global__ void __launch_bounds__(kThreads, 2)
chunk_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmU,
                const __grid_constant__ CUtensorMap tmT, const Params p) {
    using L = Smem<C, NB>;
    constexpr int NBP = L::NBP;
    constexpr int PC = C / 2;
    constexpr int CPR = C / 8;   // 16-byte chunks of a packed bf16 row
    constexpr int CPRF = C / 4;  // 16-byte chunks of an fp32 row
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sK = smem + L::kK;
    uint8_t* sV = smem + L::kV;
    uint8_t* sEB = smem + L::kEB;
    float* sSH = reinterpret_cast<float*>(smem + L::kSH);
    float* sRB = reinterpret_cast<float*>(smem + L::kRB);
    float* sbeta = reinterpret_cast<float*>(smem + L::kBeta);
    float* sg = reinterpret_cast<float*>(smem + L::kG);

    __shared__ uint64_t bar_k, bar_v, bar_mma;
    __shared__ uint32_t tmem_base_s;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
#ifdef GDN_TRACE
    int trace_n = 0;
#endif

    if (tid == 0) {
        mbar_init(&bar_k, 1);
        mbar_init(&bar_v, 1);
        mbar_init(&bar_mma, 1);
        mbar_fence_init();
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
        tma_prefetch_desc(&tmW);
        tma_prefetch_desc(&tmU);
        tma_prefetch_desc(&tmT);
    }
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_s;

    const int N = p.N, S = p.S;
    // width of the band kept in fp32 (lb[]): the order N, or all of NB for forward substitution
    const int n_band = (MODE == INV_NEUMANN) ? N : NB;
    const uint32_t n_tiles = static_cast<uint32_t>(p.n_tiles);

    // Thread t owns tile row t. Thread 0 also issues every TMA load and every tcgen05.mma, right after the
    // CTA barrier that says all rows of the operand are in place.
    const int t = tid;
    const int il = t % C;   // row inside its chunk
    const int cb = t - il;  // first tile row of the chunk
    const int wrow0 = t - lane;
    const uint32_t lane_base = tmem + (static_cast<uint32_t>(warp * 32) << 16);
    const uint32_t scratch_a = smem_u32(smem + L::kEB);
    const uint32_t br_row = smem_u32(smem + L::kBR) + t * (2 * C);
    const uint32_t sK_a = smem_u32(sK), sV_a = smem_u32(sV), sEB_a = smem_u32(sEB);
    const uint32_t idesc_g = instr_desc(128, 128, 1, 1, 0, 0, 1);
    const uint32_t idesc_c = instr_desc(128, C, 1, 1, 0, 1, 1);
    const uint32_t idesc_w = instr_desc(128, 128, 1, 1, 0, 1, 1);
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
    if (t == 0 && blockIdx.x < n_tiles) {
        const TileCoord c = decode_tile(blockIdx.x, p);
        mbar_arrive_expect_tx(&bar_k, 32768);
        tma_load_3d(sK, &tmK, &bar_k, 0, c.t0, c.bhk);
        tma_load_3d(sK + 16384, &tmK, &bar_k, 64, c.t0, c.bhk);
        mbar_arrive_expect_tx(&bar_v, 32768);
        tma_load_3d(sV, &tmV, &bar_v, 0, c.t0, c.bhv);
        tma_load_3d(sV + 16384, &tmV, &bar_v, 64, c.t0, c.bhv);
    }

    // beta and g of the row are fetched one tile ahead
    float bi_next = 0.f, gi_next = 0.f;
    if (blockIdx.x < n_tiles) {
        const TileCoord c = decode_tile(blockIdx.x, p);
        if (c.t0 + t < p.T) {
            const long long r = (long long)c.bhv * p.T + c.t0 + t;
            bi_next = __ldg(p.beta + r);
            gi_next = __ldg(p.g + r);
        }
    }

    for (uint32_t tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const TileCoord tc = decode_tile(tile, p);
        const uint32_t next = tile + gridDim.x;
        const bool has_next = next < n_tiles;
        const bool row_valid = (tc.t0 + t) < p.T;
        const long long grow = (long long)tc.bhv * p.T + tc.t0 + t;  // global token row (value-head space)

        STAMP(1);
        const float bi = bi_next, gi_ = gi_next;  // loaded during the previous tile
        // the previous tile's bulk stores have finished reading the staging slices
        if (lane == 0) tma_store_wait_read<0>();
        tc_fence_before_sync();
        compute_barrier();  // everyone is done with the previous tile's shared arrays and accumulators
        if (t == 0) {
            // G = K K^T into R0..R1 (128 columns)
            if (!wait_bar(&bar_k, par_kv)) ok = false;
            if (ok) {
                tc_fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t d = smem_desc(sK_a + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024, SWZ_128B);
                    mma_f16_ss(tmem + kR0, d, d, idesc_g, ks > 0);
                }
                mma_commit(&bar_mma);
            }
        }
        sbeta[t] = bi;
        sg[t] = gi_;
#pragma unroll
        for (int e = 0; e < NBP; ++e) sSH[t * NBP + e] = 0.f;
        if (t < 8) {
#pragma unroll
            for (int e = 0; e < NBP; ++e) sSH[(kTile + t) * NBP + e] = 0.f;
        }
        compute_barrier();

        STAMP(2);
        // ---- A-build: row of Abar from the Gram block in TMEM
        if (!wait_bar(&bar_mma, par_mma)) { ok = false; break; }
        par_mma ^= 1;
        STAMP(3);
        tc_fence_after_sync();
        float a[C];
        load_diag_block<C>(lane_base, kR0, t, a);
        {
            const float gs = gi_ * kLog2e;
            const float nbi = -bi;
            const float4* sg4 = reinterpret_cast<const float4*>(sg + cb);
#pragma unroll
            for (int j4 = 0; j4 < C / 4; ++j4) {
                const float4 gq = sg4[j4];
                const float gj[4] = {gq.x, gq.y, gq.z, gq.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int j = j4 * 4 + q;
                    const float v = nbi * fast_exp2(fmaf(-gj[q], kLog2e, gs)) * a[j];
                    a[j] = (j < il) ? v : 0.f;
                }
            }
        }

        bi_next = 0.f;
        gi_next = 0.f;
        if (has_next) {
            const TileCoord nc = decode_tile(next, p);
            if (nc.t0 + t < p.T) {
                const long long r = (long long)nc.bhv * p.T + nc.t0 + t;
                bi_next = __ldg(p.beta + r);
                gi_next = __ldg(p.g + r);
            }
        }
        STAMP(4);
        float lb[NB + 1];  // lb[d] = L[i][i-d], the band of T0 - I (or of T - I after forward substitution)
#pragma unroll
        for (int e = 0; e <= NB; ++e) lb[e] = 0.f;

        const uint32_t rowf = scratch_a + t * (4 * C);  // private fp32 row
        if constexpr (MODE == INV_NEUMANN) {
            // ---- ab[e] = Abar[i][i-e] through the private fp32 row
            float ab[NB + 1];
#pragma unroll
            for (int c = 0; c < CPRF; ++c)
                sts128(rowf + (swz<CPRF>(t, c) << 4), __float_as_uint(a[c * 4 + 0]), __float_as_uint(a[c * 4 + 1]),
                       __float_as_uint(a[c * 4 + 2]), __float_as_uint(a[c * 4 + 3]));
            ab[0] = 0.f;
#pragma unroll
            for (int e = 1; e <= NB; ++e) {
                const int j = il - e;
                ab[e] = (j >= 0) ? lds32f(rowf + (swz<CPRF>(t, j >> 2) << 4) + (j & 3) * 4) : 0.f;
            }
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
            // column form: SH[j][e-1] = L[j+e][j]
#pragma unroll
            for (int e = 1; e <= NB; ++e)
                if (il - e >= 0) sSH[(t - e) * NBP + (e - 1)] = lb[e];
            compute_barrier();

            STAMP(5);
            // ---- E = Abar + Abar L on i-j > N (in place over a[])
#pragma unroll
            for (int j = 0; j < C; ++j) {
                float v = a[j];
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
                a[j] = (il - j > N) ? v : 0.f;
            }
            // E as B operand (MN-major, no swizzle): 16-byte chunk c of row t at c * 2048 + t * 16
            if (S >= 1) {
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
        } else {
            // ---- forward substitution (Eq. 2-3). The private fp32 rows hold Abar; thread = column il of its chunk.
#pragma unroll
            for (int c = 0; c < CPRF; ++c)
                sts128(rowf + (swz<CPRF>(t, c) << 4), __float_as_uint(a[c * 4 + 0]), __float_as_uint(a[c * 4 + 1]),
                       __float_as_uint(a[c * 4 + 2]), __float_as_uint(a[c * 4 + 3]));
            compute_barrier();
            float xcol[C];  // xcol[k] = T[k][il]
#pragma unroll
            for (int i = 0; i < C; ++i) {
                float acc = 0.f;
                const uint32_t ri = scratch_a + (cb + i) * (4 * C);
#pragma unroll
                for (int k4 = 0; k4 < (i + 3) / 4; ++k4) {
                    const uint4 q = lds128(ri + (swz<CPRF>(i, k4) << 4));  // (cb + i) and i agree in the swizzle bits
                    if (k4 * 4 + 0 < i) acc = fmaf(__uint_as_float(q.x), xcol[k4 * 4 + 0], acc);
                    if (k4 * 4 + 1 < i) acc = fmaf(__uint_as_float(q.y), xcol[(k4 * 4 + 1 < C) ? k4 * 4 + 1 : 0], acc);
                    if (k4 * 4 + 2 < i) acc = fmaf(__uint_as_float(q.z), xcol[(k4 * 4 + 2 < C) ? k4 * 4 + 2 : 0], acc);
                    if (k4 * 4 + 3 < i) acc = fmaf(__uint_as_float(q.w), xcol[(k4 * 4 + 3 < C) ? k4 * 4 + 3 : 0], acc);
                }
                xcol[i] = (i > il) ? acc : ((i == il) ? 1.f : 0.f);
            }
            compute_barrier();  // everyone has read Abar
#pragma unroll
            for (int i = 0; i < C; ++i) {
                const uint32_t addr = scratch_a + (cb + i) * (4 * C) + (swz<CPRF>(i, il >> 2) << 4) + (il & 3) * 4;
                asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(xcol[i]) : "memory");
            }
            compute_barrier();
            // back to rows: a[] = far part, lb[] = band part
#pragma unroll
            for (int c = 0; c < CPRF; ++c) {
                const uint4 q = lds128(rowf + (swz<CPRF>(t, c) << 4));
                a[c * 4 + 0] = __uint_as_float(q.x);
                a[c * 4 + 1] = __uint_as_float(q.y);
                a[c * 4 + 2] = __uint_as_float(q.z);
                a[c * 4 + 3] = __uint_as_float(q.w);
            }
#pragma unroll
            for (int e = 1; e <= NB; ++e) {
                const int j = il - e;
                lb[e] = (j >= 0) ? lds32f(rowf + (swz<CPRF>(t, j >> 2) << 4) + (j & 3) * 4) : 0.f;
            }
#pragma unroll
            for (int j = 0; j < C; ++j) a[j] = (il - j > NB) ? a[j] : 0.f;
            compute_barrier();  // the fp32 rows are dead; the packed rows may overwrite them
        }

        STAMP(6);
        // ---- packed bf16 forms of the band: keep-mask (0 on the band and diagonal) and I + L
        uint32_t keep[PC], bpT[PC];
        {
            uint16_t vals[NB + 1];
#pragma unroll
            for (int e = 0; e <= NB; ++e) vals[e] = 0xFFFFu;
            build_band_row<C, NB>(br_row, t, il, n_band, vals, keep);
#pragma unroll
            for (int i = 0; i < PC; ++i) keep[i] = ~keep[i];
            vals[0] = 0x3F80u;  // 1.0
#pragma unroll
            for (int e = 1; e <= NB; ++e) vals[e] = bf16_bits(lb[e]);
            build_band_row<C, NB>(br_row, t, il, n_band, vals, bpT);
        }

        STAMP(7);
        if constexpr (MODE == INV_NEUMANN) {
            // ---- residual rounds: A_k = T0 + Z_k (bf16, TMEM), Z_{k+1} = A_k E, so that T = T0 + Z_S
            for (int k = 0; k < S; ++k) {
                uint32_t pk[PC];
                if (k == 0) {
#pragma unroll
                    for (int i = 0; i < PC; ++i) pk[i] = bpT[i];
                } else {
#pragma unroll
                    for (int i = 0; i < PC; ++i) pk[i] = (pack_bf16x2(a[2 * i], a[2 * i + 1]) & keep[i]) | bpT[i];
                }
                store_a_operand<C, false>(lane_base + kAS, t, pk);
                fence_proxy_async_smem();
                tmem_wait_st();
                tc_fence_before_sync();
                compute_barrier();
                if (t == 0) {
                    tc_fence_after_sync();
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint64_t bd = smem_desc(sEB_a + ks * 256, 128, 2048, SWZ_NONE);
                        mma_f16_ts(tmem + kR2, tmem + kAS + ks * 8, bd, idesc_c, ks > 0);
                    }
                    mma_commit(&bar_mma);
                }
                if (!wait_bar(&bar_mma, par_mma)) { ok = false; break; }
                par_mma ^= 1;
                tc_fence_after_sync();
                load_cols<C>(lane_base, kR2, a);
            }
            if (!ok) break;
            if (S == 0) {
#pragma unroll
                for (int j = 0; j < C; ++j) a[j] = 0.f;
            }
        }
        // a[] = far row (T - I - L)

        STAMP(9);
        // ---- A operands for W/U: T diag(beta) = hi + lo, hi over the whole row, lo only on band + diagonal
        {
            float tb[NB + 1];
            tb[0] = bi;
#pragma unroll
            for (int e = 1; e <= NB; ++e) tb[e] = (il - e >= 0) ? lb[e] * sbeta[(t - e) > 0 ? (t - e) : 0] : 0.f;
            uint16_t hi[NB + 1], lo[NB + 1];
#pragma unroll
            for (int e = 0; e <= NB; ++e) {
                hi[e] = bf16_bits(tb[e]);
                lo[e] = bf16_bits(tb[e] - bf16_bits_to_f32(hi[e]));
            }
            uint32_t bp[PC], pk[PC];
            build_band_row<C, NB>(br_row, t, il, n_band, hi, bp);
            const float2* sb2 = reinterpret_cast<const float2*>(sbeta + cb);
#pragma unroll
            for (int i = 0; i < PC; ++i) {
                const float2 bb = sb2[i];
                pk[i] = (pack_bf16x2(a[2 * i] * bb.x, a[2 * i + 1] * bb.y) & keep[i]) | bp[i];
            }
            store_a_operand<C, false>(lane_base + kAS, t, pk);
            build_band_row<C, NB>(br_row, t, il, n_band, lo, bp);
            store_a_operand<C, true>(lane_base + kR2, t, bp);
            tmem_wait_st();
            tc_fence_before_sync();
            compute_barrier();
        }
        if (t == 0) {
            // W = (hi + lo) K: A operands in TMEM (AS: high bf16 half, R2: low half of the band),
            // B = the K tile read as an MN-major operand (both 64-column sub-tiles, N = 128)
            tc_fence_after_sync();
#pragma unroll
            for (int ks = 0; ks < 16; ++ks) {
                const uint64_t bd = smem_desc(sK_a + (ks & 7) * 2048, 16384, 1024, SWZ_128B);
                mma_f16_ts(tmem + kR0, tmem + ((ks < 8) ? kAS : kR2) + (ks & 7) * 8, bd, idesc_w, ks > 0);
            }
            mma_commit(&bar_mma);
        }

        STAMP(8);
        // ---- T row -> Tinv: the thread's private packed row already has the TMA swizzle layout; one bulk
        // tensor store of 32 rows per warp, overlapping the W products
        if (p.Tinv != nullptr) {
#pragma unroll
            for (int c = 0; c < CPR; ++c) {
                sts128(br_row + (swz<CPR>(t, c) << 4),
                       (pack_bf16x2(a[c * 8 + 0], a[c * 8 + 1]) & keep[c * 4 + 0]) | bpT[c * 4 + 0],
                       (pack_bf16x2(a[c * 8 + 2], a[c * 8 + 3]) & keep[c * 4 + 1]) | bpT[c * 4 + 1],
                       (pack_bf16x2(a[c * 8 + 4], a[c * 8 + 5]) & keep[c * 4 + 2]) | bpT[c * 4 + 2],
                       (pack_bf16x2(a[c * 8 + 6], a[c * 8 + 7]) & keep[c * 4 + 3]) | bpT[c * 4 + 3]);
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                tma_store_3d(&tmT, smem + L::kBR + wrow0 * (2 * C), 0, tc.t0 + wrow0, tc.bhv);
                tma_store_commit();
            }
        }

        STAMP(10);
        // ---- W, then U: accumulator rows -> bf16 -> swizzled staging slice of the warp -> bulk tensor store
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
            if (!wait_bar(&bar_mma, par_mma)) { ok = false; break; }
            par_mma ^= 1;
            tc_fence_after_sync();
            STAMP(11 + half * 3);
            if (t == 0 && has_next) {
                // the products that read this tile's K (half 0) or V (half 1) are complete: prefetch the next tile's
                const TileCoord nc = decode_tile(next, p);
                if (half == 0) {
                    mbar_arrive_expect_tx(&bar_k, 32768);
                    tma_load_3d(sK, &tmK, &bar_k, 0, nc.t0, nc.bhk);
                    tma_load_3d(sK + 16384, &tmK, &bar_k, 64, nc.t0, nc.bhk);
                } else {
                    mbar_arrive_expect_tx(&bar_v, 32768);
                    tma_load_3d(sV, &tmV, &bar_v, 0, nc.t0, nc.bhv);
                    tma_load_3d(sV + 16384, &tmV, &bar_v, 64, nc.t0, nc.bhv);
                }
            }
            uint32_t o[64];
#pragma unroll
            for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(lane_base + kR0 + c0, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) o[c0 / 2 + i] = pack_bf16x2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
            }
            if (half == 0) {
                // the Tinv store of this warp has been read (the staging slices below overlap other warps' rows)
                if (lane == 0) tma_store_wait_read<0>();
                tc_fence_before_sync();
                compute_barrier();  // every row of the W accumulator has been read
                if (t == 0) {
                    if (!wait_bar(&bar_v, par_kv)) ok = false;
                    if (ok) {
                        tc_fence_after_sync();
#pragma unroll
                        for (int ks = 0; ks < 16; ++ks) {
                            const uint64_t bd = smem_desc(sV_a + (ks & 7) * 2048, 16384, 1024, SWZ_128B);
                            mma_f16_ts(tmem + kR0, tmem + ((ks < 8) ? kAS : kR2) + (ks & 7) * 8, bd, idesc_w, ks > 0);
                        }
                        mma_commit(&bar_mma);
                    }
                }
            }
            STAMP(12 + half * 3);
            {
                // the warp's 32 rows as two [32][64] sub-tiles in the 128-byte TMA swizzle, 8 KB per warp
                const uint32_t slice = scratch_a + warp * 8192;
                if (lane == 0) tma_store_wait_read<0>();  // earlier stores from this slice have been read
                __syncwarp();
#pragma unroll
                for (int c = 0; c < 16; ++c)
                    sts128(slice + (c >> 3) * 4096 + lane * 128 + (((c & 7) ^ (lane & 7)) << 4), o[c * 4 + 0], o[c * 4 + 1],
                           o[c * 4 + 2], o[c * 4 + 3]);
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    const CUtensorMap* tm = (half == 0) ? &tmW : &tmU;
                    uint8_t* src = smem + L::kEB + warp * 8192;
                    tma_store_3d(tm, src, 0, tc.t0 + wrow0, tc.bhv);
                    tma_store_3d(tm, src + 4096, 64, tc.t0 + wrow0, tc.bhv);
                    tma_store_commit();
                }
            }
            STAMP(13 + half * 3);
        }
        par_kv ^= 1;
    }
    if (lane == 0) tma_store_wait_all<0>();
    if (!ok) atomicExch(p.status, GDN_ERR_TIMEOUT);

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
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

// [heads][T][cols] bf16 tensor, boxes of `box_rows` rows x `box_cols` columns with the given swizzle
bool make_map(CUtensorMap* tm, const void* base, long long heads, int T, int cols, int box_cols, int box_rows,
              CUtensorMapSwizzle swizzle) {
    EncodeTiledFn enc = get_encode_fn();
    if (enc == nullptr) return false;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(T), static_cast<cuuint64_t>(heads)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(cols) * 2, static_cast<cuuint64_t>(T) * cols * 2};
    cuuint32_t box[3] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(box_rows), 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct Maps {
    CUtensorMap K, V, W, U, T;
};

template <int C, int NB, int MODE>
int launch_one(const Maps& m, const Params& prm, cudaStream_t stream) {
    using L = Smem<C, NB>;
    const int smem = L::kTotal + 1024;
    auto kern = chunk_tc_kernel<C, NB, MODE>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return GDN_ERR_LAUNCH;
    long long grid = prm.n_tiles < 2 * 148 ? prm.n_tiles : 2 * 148;
    kern<<<static_cast<int>(grid), kThreads, smem, stream>>>(m.K, m.V, m.W, m.U, m.T, prm);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_LAUNCH;
}

template <int C, int MODE>
int launch_c(const Maps& m, const Params& prm, cudaStream_t stream) {
    if (MODE != INV_NEUMANN || prm.N <= 3) return launch_one<C, 3, MODE>(m, prm, stream);
    return launch_one<C, 7, MODE>(m, prm, stream);
}

}  // namespace

#ifdef GDN_TRACE
extern "C" int gdn_debug_read_trace(long long* host_out) {
    return cudaMemcpyFromSymbol(host_out, g_trace, sizeof(long long) * 4096) == cudaSuccess ? 0 : -1;
}
#endif

int launch_tc_bf16(const Problem& p, InverseMode mode, cudaStream_t stream) {
    if (p.d_k != kD || p.d_v != kD) return GDN_ERR_UNSUPPORTED;
    if (!(p.C == 16 || p.C == 32 || p.C == 64)) return GDN_ERR_UNSUPPORTED;
    if (mode == INV_NEUMANN && (p.order < 1 || p.order > 7)) return GDN_ERR_UNSUPPORTED;
    if (mode == INV_FWDSUBST_BLOCKED) return GDN_ERR_UNSUPPORTED;
    if ((long long)p.B * p.H_v * p.T == 0) return GDN_OK;
    int* status = device_status_word();
    if (status == nullptr) return GDN_ERR_LAUNCH;
    Maps m;
    const long long hk = (long long)p.B * p.H_k, hv = (long long)p.B * p.H_v;
    const CUtensorMapSwizzle tsw = (p.C == 64) ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : (p.C == 32) ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
    if (!make_map(&m.K, p.K, hk, p.T, kD, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B)) return GDN_ERR_LAUNCH;
    if (!make_map(&m.V, p.V, hv, p.T, kD, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B)) return GDN_ERR_LAUNCH;
    if (!make_map(&m.W, p.W, hv, p.T, kD, 64, 32, CU_TENSOR_MAP_SWIZZLE_128B)) return GDN_ERR_LAUNCH;
    if (!make_map(&m.U, p.U, hv, p.T, kD, 64, 32, CU_TENSOR_MAP_SWIZZLE_128B)) return GDN_ERR_LAUNCH;
    // Tinv rows are C wide; without a Tinv output the map points at W (never used by the kernel then)
    if (!make_map(&m.T, p.Tinv != nullptr ? p.Tinv : p.W, hv, p.T, p.Tinv != nullptr ? p.C : kD, p.Tinv != nullptr ? p.C : 64, 32,
                  p.Tinv != nullptr ? tsw : CU_TENSOR_MAP_SWIZZLE_128B))
        return GDN_ERR_LAUNCH;
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
    if (prm.n_tiles >= (1LL << 31) - 4096 || (long long)p.B * p.H_v >= (1LL << 31)) return GDN_ERR_UNSUPPORTED;
    if (mode == INV_NEUMANN) {
        switch (p.C) {
            case 16: return launch_c<16, INV_NEUMANN>(m, prm, stream);
            case 32: return launch_c<32, INV_NEUMANN>(m, prm, stream);
            default: return launch_c<64, INV_NEUMANN>(m, prm, stream);
        }
    }
    switch (p.C) {
        case 16: return launch_c<16, INV_FWDSUBST_ROWS>(m, prm, stream);
        case 32: return launch_c<32, INV_FWDSUBST_ROWS>(m, prm, stream);
        default: return launch_c<64, INV_FWDSUBST_ROWS>(m, prm, stream);
    }
}

}  // namespace gdn
