// INT8 variant of the chunk-prepare path on the tensor cores (tcgen05 kind::i8, int32 accumulators in TMEM).
//
// Every tensor of the chain is int8 mantissas in [-127, 127] with one power-of-two exponent per chunk; the
// exponent of each requantised tensor comes from the bit length of the largest magnitude on its structural
// support (CTA-wide OR reduction per chunk), so the result is a pure function of the integer inputs and can be
// compared bit for bit with an exact-integer evaluation on the CPU. The paper fixes the uniform symmetric
// quantiser (App. G, Eq. 32), one scale per tensor, N <= 3 with residual correction (Sec. 3.5) and the band
// mask (Sec. 3.3); where quantisation is re-applied and how scales are chosen is this build's reading:
//
//   rsr(x, r)  = sign(x) ((|x| + 2^(r-1)) >> r)
//   Q8(acc, e) : r = max(0, bitlen(max |acc| on the support) - 7); q = clamp(rsr(acc, r), +-127); exponent e + r
//   align(..)  : e_ref = max(min e, max e - 8); terms shifted to e_ref (left shift, or rsr) and summed (fits int32)
//
//   G = Kq Kq^T                                   MMA (K tile by TMA, 128-byte swizzle)
//   Aq   = Q8(-(G o c), 2 k_exp - 15),  c = (beta_q_i Gam_ij + 2^14) >> 15, Gam from a 256-entry table of 2^(-f/256)
//   P_n  = Q8(band(P_{n-1} band(Aq))), n = 2..N;  T0q = Q8(align(P_1..P_N))                      integer ALU, band only
//   Eq   = Q8(align(Aq, Aq T0q)) on i-j > N                                                       integer ALU
//   R_1 = Eq, R_s = Q8(R_{s-1} Eq) on i-j >= s(N+1)                                               MMA per power
//   Sq   = Q8(align(R_1..));  Toffq = Q8(align(T0q, Sq, T0q Sq));  Tbq = Q8(Toffq_ij beta_q_j)    integer ALU
//   Wq   = Q8(align(Tbq Kq, beta_q_i Kq_i)), Uq likewise                                          MMA + ALU
//
// Work item, thread mapping, barriers and stores follow the bf16 kernel: tile of 128 tokens (two 64-chunks),
// threads t and t + 128 share tile row t and split its 64 chunk columns, thread 0 issues TMA and MMAs.
#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace gdn {
namespace {

using namespace sm100;

constexpr int kTile = 128;
constexpr int kNT = 2;                // threads per tile row (they split its 64 chunk columns and its 128 features); 4 also works
constexpr int kThreads = 128 * kNT;
constexpr int kD = 128;
constexpr int kC = 64;                // chunk size handled by this kernel
constexpr int kHC = kC / kNT;         // chunk columns per thread
constexpr int kW = kHC / 4;           // packed int8 words of a thread's part of a chunk row
constexpr int kFW = kD / kNT;         // features per thread in the W / U stage
constexpr int kNB = kHC / 8;          // blocks of eight columns per thread
constexpr int kSMax = 8;   // largest number of residual terms held in registers
constexpr int kAlignWindow = 8;  // bits kept below the largest term of an aligned sum: every such sum fits 32 bits
constexpr uint32_t kR0 = 0, kAS = 128, kTmemCols = 256;


struct ParamsI8 {
    const int16_t* beta_q;
    const int32_t* decay_q;
    const int32_t* k_exp;
    const int32_t* v_exp;
    int32_t* w_exp;
    int32_t* u_exp;
    int32_t* t_exp;
    int8_t* Toff;  // may be null
    int32_t* dbg;  // may be null: [heads * chunks][64][8 * 64 + 128 + 128] accumulators
    int* status;
    int H_k, H_v, T, group, n_tt;
    int N, S;
    int merge;     // 1: the tile is one chunk of 128 tokens whose two 64-blocks this kernel treats as chunks (see below)
    int8_t* Wq;    // raw output pointers (the block-merge kernel stores rows directly)
    int8_t* Uq;
    long long n_tiles;
    uint16_t lut[256];
};

// shared memory map (bytes)
constexpr int kOffK = 0;                 // 16 KB int8 K tile, 128-byte swizzle
constexpr int kOffV = 16384;             // 16 KB int8 V tile
constexpr int kOffEB = 32768;            // 8 KB: Eq as B operand [64 x 128] (MN-major, no swizzle)
constexpr int kOffRowA = 40960;          // 8 KB: one private 64-byte row per tile row (Aq bytes, later Sq bytes)
constexpr int kOffStage = 49152;         // 24 KB: staging of Toff (8 KB) and of W / U (4 warps x 2 halves x 2 KB)
constexpr int kOffSH = 73728;            // column form of T0q: [128 + 8][4] int
constexpr int kOffAB = kOffSH + 136 * 16;  // row form: Aq next to the diagonal / P2q: [128][8] int
constexpr int kOffBeta = kOffAB + 128 * 32;
constexpr int kOffDecay = kOffBeta + 512;
constexpr int kOffLut = kOffDecay + 512;
constexpr int kOffRed = kOffLut + 512;     // OR-reduction slots: [24][2 chunks][2 words]
constexpr int kNumRed = 24;
constexpr int kSmemTotal = kOffRed + kNumRed * 16;

__device__ __forceinline__ void cta_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory"); }

__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t i = 0;
    while (!mbar_try_wait_hint(bar, parity, 2000u)) {
        if ((++i & 63u) == 0 && clock64() - t0 > 2000000000LL) return false;
    }
    return true;
}

// rsr(x, r): rounded right shift, half away from zero; 32-bit form without branches (see rsr_rnd)
__device__ __forceinline__ int rsr32(int x, int r) {
    const int half = static_cast<int>((1u << r) >> 1);
    const int neg1 = (r > 0) ? (x >> 31) : 0;
    return (x + half + neg1) >> r;
}
// One term of an aligned sum: x 2^s for s >= 0, rounded right shift otherwise. x fits 23 bits, so the right
// shift is done in 32 bits (a shift of 31 or more gives 0, as the rounding rule demands for |x| < 2^30).
__device__ __forceinline__ int term32(int x, int s) {
    if (s >= 0) return x << s;
    return rsr32(x, (-s) < 31 ? (-s) : 31);
}
// Rounding constants of one requantisation (uniform over a chunk): shift, rounding half, and a flag that is 1 when
// something is shifted out.
struct Rnd {
    int r, half, flag;
};
__device__ __forceinline__ Rnd make_rnd(int r) {
    Rnd q;
    q.r = r;
    q.half = static_cast<int>((1u << r) >> 1);
    q.flag = (r > 0) ? 1 : 0;
    return q;
}
// rsr(x, r), branch-free: for x < 0 the rounded magnitude shift equals the arithmetic shift of x + half - 1
// (floor((x + h - 1) / 2^r) = -floor((|x| + h) / 2^r) because 2^r - h = h); r = 0 gives x.
// The correction term half - [x < 0] is one multiply-add on the (otherwise idle) multiplier pipe: the high word of
// x * flag is -1 for x < 0 and 0 otherwise (flag = 1; flag = 0 when nothing is shifted out).
__device__ __forceinline__ int mad_hi(int a, int b, int c) {
    int d;
    asm("mad.hi.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ int rsr_rnd(int x, const Rnd& q) { return (x + mad_hi(x, q.flag, q.half)) >> q.r; }
// largest magnitude of a set of values, two at a time with three-input min / max; only its bit length is used
struct MaxMag {
    int mx = 0, mn = 0;
    __device__ __forceinline__ void add2(int a, int b) {
        mx = __vimax3_s32(mx, a, b);
        mn = __vimin3_s32(mn, a, b);
    }
    __device__ __forceinline__ uint32_t mag() const { return static_cast<uint32_t>(max(mx, -mn)); }
};
// clamp(rsr(x, r), +-127)
__device__ __forceinline__ int q8_32(int x, const Rnd& q) { return max(min(rsr_rnd(x, q), 127), -127); }
__device__ __forceinline__ int q8_32(int x, int r) { return q8_32(x, make_rnd(r)); }
// cvt.pack.sat.s8.s32.b32: d[7:0] = sat8(b), d[15:8] = sat8(a), d[31:16] = c[15:0]
__device__ __forceinline__ uint32_t pack_sat_s8(int a, int b, uint32_t c) {
    uint32_t d;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// four requantised values as one word of int8: the lower clamp (-127) is explicit, the upper one (127) is the
// saturation of the pack (rsr never exceeds 128 in magnitude here)
__device__ __forceinline__ uint32_t q8_pack4(int x0, int x1, int x2, int x3, const Rnd& q) {
    const int y0 = max(rsr_rnd(x0, q), -127), y1 = max(rsr_rnd(x1, q), -127);
    const int y2 = max(rsr_rnd(x2, q), -127), y3 = max(rsr_rnd(x3, q), -127);
    return pack_sat_s8(y1, y0, pack_sat_s8(y3, y2, 0u));
}
__device__ __forceinline__ uint32_t abs32(int x) { return static_cast<uint32_t>(abs(x)); }

__device__ __forceinline__ int q8_shift(int bitlen) { return bitlen > 7 ? bitlen - 7 : 0; }
__device__ __forceinline__ int align_ref2(int e0, int e1) {
    const int lo = e0 < e1 ? e0 : e1, hi = e0 < e1 ? e1 : e0;
    return lo > hi - kAlignWindow ? lo : hi - kAlignWindow;
}
// prmt.b32 in its default mode: nibble n of `sel` picks the source byte of result byte n (0-3 from a, 4-7 from b);
// bit 3 of the nibble replicates that byte's sign bit instead of copying the byte
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
// low bytes of four ints -> one word (three byte permutes)
__device__ __forceinline__ uint32_t pack4(int a, int b, int c, int d) {
    const uint32_t ab = prmt(static_cast<uint32_t>(a), static_cast<uint32_t>(b), 0x0040u);
    const uint32_t cd = prmt(static_cast<uint32_t>(c), static_cast<uint32_t>(d), 0x0040u);
    return prmt(ab, cd, 0x5410u);
}
// byte i of w, sign-extended (one byte permute: selector 8|i replicates the sign of byte i)
__device__ __forceinline__ int byte_at(uint32_t w, int i) {
    const uint32_t sx = 8u | static_cast<uint32_t>(i);
    return static_cast<int>(prmt(w, 0u, (sx << 12) | (sx << 8) | (sx << 4) | static_cast<uint32_t>(i)));
}

// shared-memory loads by 32-bit shared address (a load through a generic pointer pays a 64-bit address computation)
__device__ __forceinline__ int lds_s32(uint32_t a) {
    int v;
    asm volatile("ld.shared.s32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ int lds_u16(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
    return static_cast<int>(v);
}
__device__ __forceinline__ int4 lds_v4(uint32_t a) {
    int4 v;
    asm volatile("ld.shared.v4.s32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a) : "memory");
    return v;
}

struct TileCoord {
    int bhk, bhv, t0;
};
__device__ __forceinline__ TileCoord decode_tile(uint32_t tile, const ParamsI8& p) {
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

// DBG: the instantiation that also dumps every tensor-core accumulator (small cases); the normal one carries none of it
template <bool DBG>
__global__ void __launch_bounds__(kThreads, 2)
chunk_tc_int8_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                     const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmU,
                     const __grid_constant__ CUtensorMap tmT, const __grid_constant__ ParamsI8 p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sK = smem + kOffK;
    uint8_t* sV = smem + kOffV;
    uint8_t* sEB = smem + kOffEB;
    uint8_t* sRowA = smem + kOffRowA;
    int* sSH = reinterpret_cast<int*>(smem + kOffSH);
    int* sAB = reinterpret_cast<int*>(smem + kOffAB);
    int* sbeta = reinterpret_cast<int*>(smem + kOffBeta);
    int* sdecay = reinterpret_cast<int*>(smem + kOffDecay);
    uint16_t* slut = reinterpret_cast<uint16_t*>(smem + kOffLut);
    uint32_t* sred = reinterpret_cast<uint32_t*>(smem + kOffRed);

    __shared__ uint64_t bar_k, bar_v, bar_mma;
    __shared__ uint32_t tmem_base_s;
    __shared__ int s_fail;  // set by warp 0 when one of its bounded waits ran out

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    if (tid == 0) {
        mbar_init(&bar_k, 1);
        mbar_init(&bar_v, 1);
        mbar_init(&bar_mma, 1);
        s_fail = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
        tma_prefetch_desc(&tmW);
        tma_prefetch_desc(&tmU);
        tma_prefetch_desc(&tmT);
    }
    if (tid < 256) slut[tid] = p.lut[tid];
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_s;

    const int N = p.N, S = p.S;
    const uint32_t n_tiles = static_cast<uint32_t>(p.n_tiles);
    const int n_c = p.T / kC;  // chunks per head

    const int t = tid & 127;        // tile row
    const int h = tid >> 7;         // which of the row's kNT threads: columns [h kHC, (h + 1) kHC)
    const int col0 = h * kHC;       // first chunk column of this thread
    const int il = t & (kC - 1);    // row inside the chunk
    const int cb = t - il;          // first tile row of the chunk
    const int ci = t >> 6;          // chunk of the tile
    const int wq = warp & 3;
    const int wrow0 = wq * 32;
    const uint32_t lane_base = tmem + (static_cast<uint32_t>(wq * 32) << 16);
    const uint32_t sK_a = smem_u32(sK), sV_a = smem_u32(sV), sEB_a = smem_u32(sEB);
    const uint32_t sdecay_a = smem_u32(sdecay), slut_a = smem_u32(slut), sSH_a = smem_u32(sSH), sbeta_a = smem_u32(sbeta);
    const uint32_t idesc_g = instr_desc(128, 128, 1, 1, 0, 0, 2);  // s8 x s8 -> s32, both K-major
    const uint32_t idesc_m = instr_desc(128, 128, 1, 1, 0, 1, 2);  // B MN-major
    uint32_t par_mma = 0, par_kv = 0;
    bool ok = true;
    // Completion of the MMAs committed to bar_mma: warp 0 polls the mbarrier, the other warps sleep on a hardware
    // barrier that warp 0 joins afterwards. A wait that ran out (here, or thread 0's waits for the K and V tiles) is
    // published in s_fail, so that all 256 threads leave the tile loop at the same point.
    auto wait_mma = [&]() -> bool {
        if (warp == 0 && (*reinterpret_cast<volatile int*>(&s_fail) != 0 || !wait_bar(&bar_mma, par_mma)))
            *reinterpret_cast<volatile int*>(&s_fail) = 1;
        asm volatile("bar.sync 2, %0;" ::"n"(kThreads) : "memory");
        par_mma ^= 1;
        return *reinterpret_cast<volatile int*>(&s_fail) == 0;
    };

    // bit length of the OR of |values| over the chunk; `slot` is a fresh reduction slot of this tile
    auto chunk_bitlen = [&](unsigned long long m, int slot) -> int {
        uint32_t lo = __reduce_or_sync(0xFFFFFFFFu, static_cast<uint32_t>(m));
        uint32_t hi = __reduce_or_sync(0xFFFFFFFFu, static_cast<uint32_t>(m >> 32));
        if (lane == 0) {
            if (lo) atomicOr(&sred[(slot * 2 + ci) * 2 + 0], lo);
            if (hi) atomicOr(&sred[(slot * 2 + ci) * 2 + 1], hi);
        }
        cta_barrier();
        const unsigned long long all =
            (static_cast<unsigned long long>(sred[(slot * 2 + ci) * 2 + 1]) << 32) | sred[(slot * 2 + ci) * 2 + 0];
        return all ? 64 - __clzll(static_cast<long long>(all)) : 0;
    };
    // the same for values known to fit 32 bits (one warp reduction, one shared-memory atomic)
    auto chunk_bitlen32 = [&](uint32_t m, int slot) -> int {
        const uint32_t lo = __reduce_or_sync(0xFFFFFFFFu, m);
        if (lane == 0 && lo) atomicOr(&sred[(slot * 2 + ci) * 2 + 0], lo);
        cta_barrier();
        const uint32_t all = sred[(slot * 2 + ci) * 2 + 0];
        return 32 - __clz(static_cast<int>(all));
    };

    if (tid == 0 && blockIdx.x < n_tiles) {
        const TileCoord c = decode_tile(blockIdx.x, p);
        mbar_arrive_expect_tx(&bar_k, 16384);
        tma_load_3d(sK, &tmK, &bar_k, 0, c.t0, c.bhk);
        mbar_arrive_expect_tx(&bar_v, 16384);
        tma_load_3d(sV, &tmV, &bar_v, 0, c.t0, c.bhv);
    }

    for (uint32_t tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const TileCoord tc = decode_tile(tile, p);
        const uint32_t next = tile + gridDim.x;
        const bool has_next = next < n_tiles;
        const bool row_valid = (tc.t0 + t) < p.T;
        const long long grow = (long long)tc.bhv * p.T + tc.t0 + t;
        const int chunk_in_head = (tc.t0 + cb) / kC;
        const bool chunk_valid = (tc.t0 + cb) < p.T;

        // row of the accumulator dump (debugging aid of small cases; null in normal use)
        constexpr int kDbgRow = 8 * kC + 2 * kD;
        int32_t* dbg_row = (DBG && p.dbg != nullptr && row_valid)
                               ? p.dbg + (((long long)tc.bhv * n_c + chunk_in_head) * kC + il) * kDbgRow
                               : nullptr;
        int bq = 0, dq = 0, kexp = 0, vexp = 0;
        if (row_valid) {
            bq = static_cast<int>(static_cast<uint16_t>(p.beta_q[grow]));
            dq = p.decay_q[grow];
        }
        if (chunk_valid) {
            // (chunks of 128 tokens: one input exponent per 128 tokens, shared by the two 64-blocks)
            const int n_ce = p.merge ? (n_c >> 1) : n_c, ce = p.merge ? (chunk_in_head >> 1) : chunk_in_head;
            kexp = p.k_exp[(long long)tc.bhk * n_ce + ce];
            vexp = p.v_exp[(long long)tc.bhv * n_ce + ce];
        }
        if (lane == 0) tma_store_wait_read<0>();
        tc_fence_before_sync();
        cta_barrier();  // previous tile finished with shared arrays and accumulators
        if (tid == 0) {
            if (!wait_bar(&bar_k, par_kv)) {
                ok = false;
                *reinterpret_cast<volatile int*>(&s_fail) = 1;
            }
            if (ok) {
                tc_fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const uint64_t d = smem_desc(sK_a + ks * 32, 16, 1024, SWZ_128B);
                    mma_i8_ss(tmem + kR0, d, d, idesc_g, ks > 0);
                }
                mma_commit(&bar_mma);
            }
        }
        if (h == 0) {
            sbeta[t] = bq;
            sdecay[t] = dq;
#pragma unroll
            for (int e = 0; e < 4; ++e) sSH[t * 4 + e] = 0;
            if (t < 8) {
#pragma unroll
                for (int e = 0; e < 4; ++e) sSH[(kTile + t) * 4 + e] = 0;
            }
        }
        if (tid < kNumRed * 4) sred[tid] = 0u;
        cta_barrier();
        int slot = 0;

        // ---- I1-I3: Aq = Q8(-(G o c))
        if (!wait_mma()) { ok = false; break; }
        tc_fence_after_sync();
        int aq[kHC];
        int eA;
        {
            uint32_t g[kHC];
            tmem_ldn(lane_base + kR0 + cb + col0, g);
            tmem_wait_ld();
            if (DBG && dbg_row != nullptr) {
#pragma unroll
                for (int jl = 0; jl < kHC; ++jl) dbg_row[col0 + jl] = static_cast<int>(g[jl]);
            }
            // c_ij = (beta_q_i Gam_ij + 2^14) >> 15 (< 2^15), 0 on and above the diagonal. |G| < 2^21, so |G| c needs
            // 36 bits: it is kept as a (hi, lo) pair of 32-bit words; the shift r = bitlen - 7 stays below 32, so the
            // rounded shift is one funnel shift of the pair. Aq = -G c: the sign is restored at the end (the rounding
            // rule is symmetric).
            int cq[kHC];
            uint32_t mlo = 0, mhi = 0;
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) {
                const int j = col0 + jl;
                const int dlt = dq - lds_s32(sdecay_a + (cb + j) * 4);
                const int sh = dlt >> 8;
                const int gam = (sh >= 0 && sh < 16) ? (lds_u16(slut_a + (dlt & 255) * 2) >> sh) : 0;
                const int c = (j < il) ? ((bq * gam + (1 << 14)) >> 15) : 0;
                cq[jl] = c;
                const uint32_t ag = static_cast<uint32_t>(abs(static_cast<int>(g[jl])));
                mlo |= ag * static_cast<uint32_t>(c);
                mhi |= __umulhi(ag, static_cast<uint32_t>(c));
            }
            const int r = q8_shift(chunk_bitlen((static_cast<unsigned long long>(mhi) << 32) | mlo, slot++));
            const uint32_t half = (1u << r) >> 1;
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) {
                const int gv = static_cast<int>(g[jl]);
                const uint32_t ag = static_cast<uint32_t>(abs(gv)), c = static_cast<uint32_t>(cq[jl]);
                const uint32_t lo = ag * c, lo2 = lo + half;
                const uint32_t hi2 = __umulhi(ag, c) + (lo2 < lo ? 1u : 0u);
                const int q = static_cast<int>(min(__funnelshift_r(lo2, hi2, r), 127u));
                aq[jl] = (gv < 0) ? q : -q;
            }
            eA = 2 * kexp - 15 + r;
        }
        // Aq bytes to the private row; entries next to the diagonal and right of this half come back from there
        uint8_t* rowa = sRowA + t * 64;
#pragma unroll
        for (int c = 0; c < kHC / 16; ++c)
            *reinterpret_cast<uint4*>(rowa + col0 + 16 * c) =
                make_uint4(pack4(aq[16 * c + 0], aq[16 * c + 1], aq[16 * c + 2], aq[16 * c + 3]),
                           pack4(aq[16 * c + 4], aq[16 * c + 5], aq[16 * c + 6], aq[16 * c + 7]),
                           pack4(aq[16 * c + 8], aq[16 * c + 9], aq[16 * c + 10], aq[16 * c + 11]),
                           pack4(aq[16 * c + 12], aq[16 * c + 13], aq[16 * c + 14], aq[16 * c + 15]));
        cta_barrier();
        int ab1 = 0, ab2 = 0, ab3 = 0;  // Aq[i][i-1..i-3]
        if (il >= 1) ab1 = static_cast<int>(static_cast<int8_t>(rowa[il - 1]));
        if (il >= 2) ab2 = static_cast<int>(static_cast<int8_t>(rowa[il - 2]));
        if (il >= 3) ab3 = static_cast<int>(static_cast<int8_t>(rowa[il - 3]));
        int an0 = 0, an1 = 0, an2 = 0;  // the three entries of the row right of this thread's columns
        if (h < kNT - 1) {
            an0 = static_cast<int>(static_cast<int8_t>(rowa[col0 + kHC + 0]));
            an1 = static_cast<int>(static_cast<int8_t>(rowa[col0 + kHC + 1]));
            an2 = static_cast<int>(static_cast<int8_t>(rowa[col0 + kHC + 2]));
        }
        // P_1 = band of Aq: zero beyond distance N
        const int p11 = ab1, p12 = (N >= 2) ? ab2 : 0, p13 = (N >= 3) ? ab3 : 0;
        if (h == 0) {
            sAB[t * 8 + 1] = p11;
            sAB[t * 8 + 2] = p12;
            sAB[t * 8 + 3] = p13;
        }
        cta_barrier();

        // ---- I4: P_2, P_3 (band only), I5: T0q
        int t0q1 = 0, t0q2 = 0, t0q3 = 0;  // T0q[i][i-1..i-3]
        int eT0;
        {
            const int r1 = (t - 1) > 0 ? (t - 1) : 0, r2 = (t - 2) > 0 ? (t - 2) : 0;
            // P_2 on distances 2..N: sum over the intermediate row
            int acc22 = (N >= 2) ? p11 * sAB[r1 * 8 + 1] : 0;
            int acc23 = (N >= 3) ? p11 * sAB[r1 * 8 + 2] + p12 * sAB[r2 * 8 + 1] : 0;
            int p22 = 0, p23 = 0, p33 = 0;
            int e2 = 0, e3 = 0;
            if (N >= 2) {
                const uint32_t m = (h == 0) ? (abs32(acc22) | abs32(acc23)) : 0u;
                const int r = q8_shift(chunk_bitlen32(m, slot++));
                p22 = q8_32(acc22, r);
                p23 = q8_32(acc23, r);
                e2 = eA + eA + r;
            }
            if (N >= 3) {
                // P_3 at distance 3: P_2[i][i-2] * Aq[i-2][i-3]
                const int acc3 = p22 * sAB[r2 * 8 + 1];
                const int r = q8_shift(chunk_bitlen32((h == 0) ? abs32(acc3) : 0u, slot++));
                p33 = q8_32(acc3, r);
                e3 = e2 + eA + r;
            }
            // align(P_1..P_N): at most three small terms per band entry
            int emin = eA, emax = eA;
            if (N >= 2) { emin = min(emin, e2); emax = max(emax, e2); }
            if (N >= 3) { emin = min(emin, e3); emax = max(emax, e3); }
            const int eref = max(emin, emax - kAlignWindow);
            const int s1 = eA - eref, s2 = e2 - eref, s3 = e3 - eref;
            int a1 = term32(p11, s1);
            int a2 = term32(p12, s1) + ((N >= 2) ? term32(p22, s2) : 0);
            int a3 = term32(p13, s1) + ((N >= 2) ? term32(p23, s2) : 0) + ((N >= 3) ? term32(p33, s3) : 0);
            if (!(N >= 1 && il >= 1)) a1 = 0;
            if (!(N >= 2 && il >= 2)) a2 = 0;
            if (!(N >= 3 && il >= 3)) a3 = 0;
            const uint32_t m = (h == 0) ? (abs32(a1) | abs32(a2) | abs32(a3)) : 0u;
            const int r = q8_shift(chunk_bitlen32(m, slot++));
            t0q1 = q8_32(a1, r);
            t0q2 = q8_32(a2, r);
            t0q3 = q8_32(a3, r);
            eT0 = eref + r;
            if (h == 0) {
                if (il >= 1) sSH[(t - 1) * 4 + 0] = t0q1;
                if (il >= 2) sSH[(t - 2) * 4 + 1] = t0q2;
                if (il >= 3) sSH[(t - 3) * 4 + 2] = t0q3;
            }
            cta_barrier();
        }

        // ---- I6: Eq = Q8(align(Aq, Aq T0q)) on i-j > N
        int eq[kHC];
        int eE;
        {
            const int eref = align_ref2(eA, eA + eT0);
            const int sa = eA - eref, sp = eA + eT0 - eref;
            int acc[kHC];  // |Aq| < 2^7 and |Aq T0q| <= 3 * 127^2 < 2^16, shifted left by at most 8
            const bool left = sa >= 0 && sp >= 0;
            uint32_t m = 0;
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) {
                const int4 c4 = lds_v4(sSH_a + (cb + col0 + jl) * 16);
                const int a1 = (jl + 1 < kHC) ? aq[(jl + 1 < kHC) ? jl + 1 : 0] : ((jl + 1 == kHC) ? an0 : (jl + 1 == kHC + 1 ? an1 : an2));
                const int a2 = (jl + 2 < kHC) ? aq[(jl + 2 < kHC) ? jl + 2 : 0] : ((jl + 2 == kHC) ? an0 : (jl + 2 == kHC + 1 ? an1 : an2));
                const int a3 = (jl + 3 < kHC) ? aq[(jl + 3 < kHC) ? jl + 3 : 0] : ((jl + 3 == kHC) ? an0 : (jl + 3 == kHC + 1 ? an1 : an2));
                const bool on = (il - (col0 + jl)) > N;
                const int pr = a1 * c4.x + a2 * c4.y + a3 * c4.z;
                const int v = on ? (left ? ((aq[jl] << sa) + (pr << sp)) : (term32(aq[jl], sa) + term32(pr, sp))) : 0;
                acc[jl] = v;
            }
            MaxMag mm;
#pragma unroll
            for (int jl = 0; jl < kHC; jl += 2) mm.add2(acc[jl], acc[jl + 1]);
            m = mm.mag();
            const int r = q8_shift(chunk_bitlen32(m, slot++));
            const Rnd rq = make_rnd(r);
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) eq[jl] = q8_32(acc[jl], rq);
            eE = eref + r;
        }
        // Rows of the powers R_s (R_1 = Eq) as packed bytes. The loops over the powers are NOT unrolled (the kernel is bound
        // by instruction fetch: its straight-line code is larger than the instruction cache), so the rows cannot sit in
        // registers indexed by s: R_1 stays in registers, R_2.. are parked in free TMEM columns of the row's own lane
        // (columns 160..255 for s = 2..7; s = 8 and, for the sum, R_1 go to accumulator columns that are idle by then).
        uint32_t r1[kHC / 4];   // R_1
        uint32_t cur[kHC / 4];  // R_{s-1} inside the loop
        int er[kSMax];
#pragma unroll
        for (int s = 0; s < kSMax; ++s) er[s] = 0;
#pragma unroll
        for (int w = 0; w < kHC / 4; ++w) r1[w] = cur[w] = 0u;
        auto park_col = [&](int s) -> uint32_t {  // TMEM column of the parked row of R_s (s >= 1)
            return (s >= 2 && s <= 7) ? static_cast<uint32_t>(160 + (s - 2) * 16 + h * kW)
                                      : static_cast<uint32_t>(kR0 + (s == 1 ? 0 : 16) + h * kW);
        };
        // Structural support: R_s is zero for i - j < s (N + 1), so of this thread's four blocks of eight columns only the
        // first live_blocks(s) can hold a non-zero entry in any of the warp's 32 rows (a warp-uniform count; the warp
        // with rows 0..31 and columns 32..63 has none at all). Dead blocks are skipped in the requantisation and in the
        // sum. With the debug output every block is walked (the test reads every accumulator).
        const int row_max = (wrow0 & (kC - 1)) + 31;
        const bool walk_all = DBG && p.dbg != nullptr;
        auto live_blocks = [&](int s) -> int {
            const int x = row_max - col0 - s * (N + 1);
            return walk_all ? kNB : (x < 0 ? 0 : min(kNB, (x >> 3) + 1));
        };
        int n_terms = 0;
        if (S >= 1) {
#pragma unroll
            for (int w = 0; w < kHC / 4; ++w) r1[w] = cur[w] = pack4(eq[4 * w], eq[4 * w + 1], eq[4 * w + 2], eq[4 * w + 3]);
            er[0] = eE;
            n_terms = 1;
            // B operand [E_1 | E_2] (64 x 128 int8, MN-major, no swizzle): 16 columns of chunk-row il per 16-byte piece
#pragma unroll
            for (int c = 0; c < kHC / 16; ++c) {
                const uint4 v = make_uint4(r1[4 * c], r1[4 * c + 1], r1[4 * c + 2], r1[4 * c + 3]);
                *reinterpret_cast<uint4*>(sEB + (((cb + col0) >> 4) + c) * (16 * kC) + il * 16) = v;
            }
        }
        // ---- I7: R_s = Q8(R_{s-1} Eq) while s (N+1) < C
#pragma unroll 1
        for (int s = 2; s <= kSMax; ++s) {
            if (s > S || s * (N + 1) >= kC) break;
            tmem_stn(lane_base + kAS + h * kW, cur);
            fence_proxy_async_smem();
            tmem_wait_st();
            tc_fence_before_sync();
            cta_barrier();
            if (tid == 0) {
                tc_fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < kC / 32; ++ks) {
                    const uint64_t bd = smem_desc(sEB_a + ks * 512, 128, 16 * kC, SWZ_NONE);
                    mma_i8_ts(tmem + kR0, tmem + kAS + ks * 8, bd, idesc_m, ks > 0);
                }
                mma_commit(&bar_mma);
            }
            if (!wait_mma()) { ok = false; break; }
            tc_fence_after_sync();
            uint32_t dres[kHC];
            tmem_ldn(lane_base + kR0 + cb + col0, dres);
            tmem_wait_ld();
            if (DBG && dbg_row != nullptr) {
#pragma unroll
                for (int jl = 0; jl < kHC; ++jl) dbg_row[(s - 1) * kC + col0 + jl] = static_cast<int>(dres[jl]);
            }
            uint32_t m = 0;
            // R_{s-1} is zero for i - j < (s - 1)(N + 1) and Eq for i - j <= N: the integer product is exactly zero
            // for i - j < s (N + 1), no mask needed
            const int nb = live_blocks(s);
            {
                MaxMag mm;
#pragma unroll
                for (int b = 0; b < kNB; ++b) {
                    if (b < nb) {
#pragma unroll
                        for (int jl = 8 * b; jl < 8 * b + 8; jl += 2) mm.add2(static_cast<int>(dres[jl]), static_cast<int>(dres[jl + 1]));
                    }
                }
                m = mm.mag();
            }
            const int r = q8_shift(chunk_bitlen32(m, slot++));  // (its barrier: every thread has read the accumulator)
            const Rnd rq = make_rnd(r);
#pragma unroll
            for (int b = 0; b < kNB; ++b) {
                cur[2 * b] = cur[2 * b + 1] = 0u;
                if (b < nb) {
#pragma unroll
                    for (int w = 2 * b; w < 2 * b + 2; ++w)
                        cur[w] = q8_pack4(static_cast<int>(dres[4 * w]), static_cast<int>(dres[4 * w + 1]),
                                          static_cast<int>(dres[4 * w + 2]), static_cast<int>(dres[4 * w + 3]), rq);
                }
            }
            tmem_stn(lane_base + park_col(s), cur);
            er[s - 1] = er[s - 2] + eE + r;
            n_terms = s;
        }
        if (!ok) break;

        // ---- Sq = Q8(align(R_1..)): the exponents fall by several bits per power, so most terms are
        // shifted far to the right; a term whose right shift exceeds 7 rounds to zero and is skipped
        int sq[kHC];
        int eS = 0;
        if (n_terms > 0) {
            int emin = er[0], emax = er[0];
#pragma unroll
            for (int s = 1; s < kSMax; ++s)
                if (s < n_terms) { emin = min(emin, er[s]); emax = max(emax, er[s]); }
            const int eref = max(emin, emax - kAlignWindow);
            int acc[kHC];
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) acc[jl] = 0;
            tmem_stn(lane_base + park_col(1), r1);
            tmem_wait_st();
#pragma unroll 1
            for (int s = 1; s <= n_terms; ++s) {
                const int sh = er[s - 1] - eref;
                if (sh < -7) continue;
                const int nb = live_blocks(s);
                if (nb == 0) continue;
                uint32_t w[kHC / 4];
                tmem_ldn(lane_base + park_col(s), w);
                tmem_wait_ld();
                if (sh >= 0) {
#pragma unroll
                    for (int b = 0; b < kNB; ++b) {
                        if (b < nb) {
#pragma unroll
                            for (int jl = 8 * b; jl < 8 * b + 8; ++jl) acc[jl] += byte_at(w[jl >> 2], jl & 3) << sh;
                        }
                    }
                } else {
#pragma unroll
                    for (int b = 0; b < kNB; ++b) {
                        if (b < nb) {
#pragma unroll
                            for (int jl = 8 * b; jl < 8 * b + 8; ++jl) acc[jl] += rsr32(byte_at(w[jl >> 2], jl & 3), -sh);
                        }
                    }
                }
            }
            const int nb1 = live_blocks(1);  // the support of the sum is that of its first term
            MaxMag mm;
#pragma unroll
            for (int b = 0; b < kNB; ++b) {
                if (b < nb1) {
#pragma unroll
                    for (int jl = 8 * b; jl < 8 * b + 8; jl += 2) mm.add2(acc[jl], acc[jl + 1]);
                }
            }
            const uint32_t m = mm.mag();
            const int r = q8_shift(chunk_bitlen32(m, slot++));
            const Rnd rq = make_rnd(r);
#pragma unroll
            for (int b = 0; b < kNB; ++b) {
#pragma unroll
                for (int jl = 8 * b; jl < 8 * b + 8; ++jl) sq[jl] = 0;
                if (b < nb1) {
#pragma unroll
                    for (int jl = 8 * b; jl < 8 * b + 8; ++jl) sq[jl] = q8_32(acc[jl], rq);
                }
            }
            eS = eref + r;
        } else {
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) sq[jl] = 0;
        }
        // Sq bytes to the private rows (the rows above are needed for T0q Sq)
#pragma unroll
        for (int c = 0; c < kHC / 16; ++c)
            *reinterpret_cast<uint4*>(rowa + col0 + 16 * c) =
                make_uint4(pack4(sq[16 * c + 0], sq[16 * c + 1], sq[16 * c + 2], sq[16 * c + 3]),
                           pack4(sq[16 * c + 4], sq[16 * c + 5], sq[16 * c + 6], sq[16 * c + 7]),
                           pack4(sq[16 * c + 8], sq[16 * c + 9], sq[16 * c + 10], sq[16 * c + 11]),
                           pack4(sq[16 * c + 12], sq[16 * c + 13], sq[16 * c + 14], sq[16 * c + 15]));
        cta_barrier();

        // ---- I8: Toffq = Q8(align(T0q, Sq, T0q Sq)) on i > j
        int toff[kHC];   // far part of the row (zero on the band)
        int tband[3];    // Toffq[i][i-1..i-3] (zero where the row or the order has no such entry)
        int eT;
        {
            int prod[kHC];
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) prod[jl] = 0;
#pragma unroll
            for (int e = 1; e <= 3; ++e) {
                const int rr = (t - e) > 0 ? (t - e) : 0;
                const int cf = (il - e >= 0) ? (e == 1 ? t0q1 : (e == 2 ? t0q2 : t0q3)) : 0;
                uint32_t w[kW];
#pragma unroll
                for (int c = 0; c < kHC / 16; ++c) {
                    const int4 a0 = lds_v4(smem_u32(sRowA) + rr * 64 + col0 + 16 * c);
                    w[4 * c] = a0.x; w[4 * c + 1] = a0.y; w[4 * c + 2] = a0.z; w[4 * c + 3] = a0.w;
                }
#pragma unroll
                for (int jl = 0; jl < kHC; ++jl) prod[jl] += cf * byte_at(w[jl >> 2], jl & 3);
            }
            const int e0 = eT0, e1 = eS, e2 = eT0 + eS;
            const int emin = min(e0, min(e1, e2)), emax = max(e0, max(e1, e2));
            const int eref = max(emin, emax - kAlignWindow);
            const int s0 = e0 - eref, s1 = e1 - eref, s2 = e2 - eref;
            // The band entries and Sq never share an element (band: distance <= N, Sq: distance > N), and Sq and T0q Sq
            // are exactly zero on the band, the diagonal and above (Sq by its support, the product because T0q is banded
            // and lower triangular). So the row's 32 columns take the far formula without any mask, and the (at most
            // three) band entries of the row are three scalars, T0q alone: entries below 2^7, the product below
            // 3 * 127^2 < 2^16. The band values are put into the packed rows afterwards, through shared memory.
            const bool left = s0 >= 0 && s1 >= 0 && s2 >= 0;
            int acc[kHC];
            uint32_t m = 0;
            if (left) {
#pragma unroll
                for (int jl = 0; jl < kHC; ++jl) acc[jl] = (sq[jl] << s1) + (prod[jl] << s2);
            } else {
#pragma unroll
                for (int jl = 0; jl < kHC; ++jl) acc[jl] = term32(sq[jl], s1) + term32(prod[jl], s2);
            }
            const int ab1 = term32(t0q1, s0), ab2 = term32(t0q2, s0), ab3 = term32(t0q3, s0);
            {
                MaxMag mm;
#pragma unroll
                for (int jl = 0; jl < kHC; jl += 2) mm.add2(acc[jl], acc[jl + 1]);
                mm.add2(ab1, ab2);
                mm.add2(ab3, 0);
                m = mm.mag();
            }
            const int r = q8_shift(chunk_bitlen32(m, slot++));
            const Rnd rq = make_rnd(r);
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) toff[jl] = q8_32(acc[jl], rq);
            tband[0] = q8_32(ab1, rq);
            tband[1] = q8_32(ab2, rq);
            tband[2] = q8_32(ab3, rq);
            eT = eref + r;
        }

        // ---- I9: Tbq = Q8(Toffq_ij beta_q_j); A operand of W/U (block diagonal, int8 in TMEM)
        int eTb;
        {
            int acc[kHC];
            uint32_t m = 0;
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) {
                acc[jl] = toff[jl] * lds_s32(sbeta_a + (cb + col0 + jl) * 4);
            }
            int accb[3];  // the band entries times beta of their columns
#pragma unroll
            for (int e = 1; e <= 3; ++e) accb[e - 1] = (il - e >= 0) ? tband[e - 1] * sbeta[t - e] : 0;
            {
                MaxMag mm;
#pragma unroll
                for (int jl = 0; jl < kHC; jl += 2) mm.add2(acc[jl], acc[jl + 1]);
                mm.add2(accb[0], accb[1]);
                mm.add2(accb[2], 0);
                m = mm.mag();
            }
            const int r = q8_shift(chunk_bitlen32(m, slot++));
            const Rnd rq9 = make_rnd(r);
            uint32_t r8[kW];
#pragma unroll
            for (int w = 0; w < kW; ++w)
                r8[w] = q8_pack4(acc[4 * w], acc[4 * w + 1], acc[4 * w + 2], acc[4 * w + 3], rq9);
            // the band bytes go in through the row's private shared-memory line (free since the reduction above: every
            // thread is past its reads of the Sq rows); a thread patches the columns it owns and reads its part back
#pragma unroll
            for (int c = 0; c < kHC / 16; ++c)
                *reinterpret_cast<uint4*>(rowa + col0 + 16 * c) = make_uint4(r8[4 * c], r8[4 * c + 1], r8[4 * c + 2], r8[4 * c + 3]);
#pragma unroll
            for (int e = 1; e <= 3; ++e) {
                const int c = il - e;
                if (e <= N && c >= col0 && c < col0 + kHC) rowa[c] = static_cast<uint8_t>(q8_32(accb[e - 1], rq9) & 0xFF);
            }
#pragma unroll
            for (int c = 0; c < kHC / 16; ++c) {
                const uint4 v = *reinterpret_cast<const uint4*>(rowa + col0 + 16 * c);
                r8[4 * c] = v.x; r8[4 * c + 1] = v.y; r8[4 * c + 2] = v.z; r8[4 * c + 3] = v.w;
            }
            eTb = eT - 15 + r;
            // row t's block occupies packed columns [cb/4, cb/4 + 16) of a 32-column operand; the other 16 are zero
            tmem_stn(lane_base + kAS + cb / 4 + h * kW, r8);
#pragma unroll
            for (int w = 0; w < kW; ++w) r8[w] = 0u;
            tmem_stn(lane_base + kAS + (16 - cb / 4) + h * kW, r8);
            tmem_wait_st();
        }
        // Toffq row -> staging (64-byte lines, 64-byte TMA swizzle) -> bulk tensor store of 32 rows per warp (h = 0 issues)
        uint8_t* stage = smem + kOffStage;
        if (p.Toff != nullptr) {
            uint8_t* line = stage + t * 64;
#pragma unroll
            for (int c = 0; c < kHC / 16; ++c) {
                const int cc = (col0 >> 4) + c;
                const uint4 v = make_uint4(pack4(toff[16 * c + 0], toff[16 * c + 1], toff[16 * c + 2], toff[16 * c + 3]),
                                           pack4(toff[16 * c + 4], toff[16 * c + 5], toff[16 * c + 6], toff[16 * c + 7]),
                                           pack4(toff[16 * c + 8], toff[16 * c + 9], toff[16 * c + 10], toff[16 * c + 11]),
                                           pack4(toff[16 * c + 12], toff[16 * c + 13], toff[16 * c + 14], toff[16 * c + 15]));
                *reinterpret_cast<uint4*>(line + ((cc ^ ((t >> 1) & 3)) << 4)) = v;
            }
#pragma unroll
            for (int e = 1; e <= 3; ++e) {
                const int c = il - e;
                if (e <= N && c >= col0 && c < col0 + kHC)
                    line[(((c >> 4) ^ ((t >> 1) & 3)) << 4) + (c & 15)] = static_cast<uint8_t>(tband[e - 1] & 0xFF);
            }
        }
        if (row_valid && il == 0 && h == 0) {
            // chunks of 128 tokens: three exponents per chunk (e11, e21, e22); this kernel writes the diagonal ones
            const long long ti = p.merge ? (((long long)tc.bhv * (n_c >> 1) + (chunk_in_head >> 1)) * 3 + 2 * (chunk_in_head & 1))
                                         : ((long long)tc.bhv * n_c + chunk_in_head);
            p.t_exp[ti] = eT;
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        cta_barrier();
        if (p.Toff != nullptr && h == 0 && lane == 0) {
            tma_store_3d(&tmT, stage + wrow0 * 64, p.merge ? ci * kC : 0, tc.t0 + wrow0, tc.bhv);
            tma_store_commit();
        }
        if (tid == 0) {
            // W accumulator = blockdiag(Tbq) Kq: M = 128, N = 128, K = 128 (4 steps of 32)
            tc_fence_after_sync();
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                const uint64_t bd = smem_desc(sK_a + ks * 4096, 16384, 1024, SWZ_128B);
                mma_i8_ts(tmem + kR0, tmem + kAS + ks * 8, bd, idesc_m, ks > 0);
            }
            mma_commit(&bar_mma);
        }

        // ---- I10: W, then U
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
            const int xexp = (half == 0) ? kexp : vexp;
            // diagonal term beta_q_i * Xq_i for this thread's 64 columns, from its own row of the int8 tile
            uint32_t xr[kFW / 4];
#pragma unroll
            for (int c = 0; c < kFW / 16; ++c) {
                const int4 v = lds_v4(((half == 0) ? sK_a : sV_a) + t * 128 + (((h * (kFW / 16) + c) ^ (t & 7)) << 4));
                xr[4 * c + 0] = v.x; xr[4 * c + 1] = v.y; xr[4 * c + 2] = v.z; xr[4 * c + 3] = v.w;
            }
            if (!wait_mma()) { ok = false; break; }
            tc_fence_after_sync();
            const int ep = eTb + xexp, ed = xexp - 15;
            const int eref = align_ref2(ep, ed);
            const int sp = ep - eref, sd = ed - eref;
            // |Tbq Xq| <= 128 * 127^2 < 2^21, |beta_q Xq| < 2^22; at most one of them is shifted left, by at most 8
            // pass 1: the scale (bit length of the largest magnitude over the chunk's C x d block)
            const bool left = sp >= 0 && sd >= 0;  // the usual case: plain left shifts
            const int psc = left ? (1 << sp) : 0, bqs = left ? (bq << sd) : 0;
            MaxMag mmw;
            int sums[kFW];  // the aligned sums of this thread's columns stay in registers between the two passes
#pragma unroll
            for (int c0 = 0; c0 < kFW; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(lane_base + kR0 + h * kFW + c0, r);
                tmem_wait_ld();
                if (DBG && dbg_row != nullptr) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) dbg_row[8 * kC + half * kD + h * kFW + c0 + i] = static_cast<int>(r[i]);
                }
                if (left) {
                    // shifts folded into the multipliers: two multiply-adds per element
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        sums[c0 + i] = static_cast<int>(r[i]) * psc + byte_at(xr[(c0 + i) >> 2], (c0 + i) & 3) * bqs;
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        sums[c0 + i] = term32(static_cast<int>(r[i]), sp) + term32(bq * byte_at(xr[(c0 + i) >> 2], (c0 + i) & 3), sd);
                }
#pragma unroll
                for (int i = 0; i < 32; i += 2) mmw.add2(sums[c0 + i], sums[c0 + i + 1]);
            }
            const int rr = q8_shift(chunk_bitlen32(mmw.mag(), slot++));
            const Rnd rqw = make_rnd(rr);
            // after that barrier every thread holds its own row of the K (V) tile in registers, and the products that
            // read the tile are complete: the next tile's K (V) may land
            if (tid == 0 && has_next) {
                const TileCoord nc = decode_tile(next, p);
                if (half == 0) {
                    mbar_arrive_expect_tx(&bar_k, 16384);
                    tma_load_3d(sK, &tmK, &bar_k, 0, nc.t0, nc.bhk);
                } else {
                    mbar_arrive_expect_tx(&bar_v, 16384);
                    tma_load_3d(sV, &tmV, &bar_v, 0, nc.t0, nc.bhv);
                }
            }
            if (row_valid && il == 0 && h == 0)
                ((half == 0) ? p.w_exp : p.u_exp)[(long long)tc.bhv * n_c + chunk_in_head] = eref + rr;
            // pass 2: mantissas. Two threads per row: 32 rows x 64 int8 columns of this warp in the 64-byte TMA swizzle
            // (2 KB at stage + 8 KB + (wq * 2 + h) * 2 KB), stored by a bulk tensor store below. Four threads per row:
            // 32 bytes of the row straight to global memory (a whole 32-byte sector per thread).
            uint8_t* sub = stage + 8192 + (wq * 2 + (h & 1)) * 2048;
            if (kNT == 2) {
                if (lane == 0) tma_store_wait_read<0>();
                __syncwarp();
            }
#pragma unroll
            for (int c0 = 0; c0 < kFW; c0 += 32) {
                const int* qv = sums + c0;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const int cc = c0 / 16 + c;
                    const uint4 v = make_uint4(q8_pack4(qv[16 * c + 0], qv[16 * c + 1], qv[16 * c + 2], qv[16 * c + 3], rqw),
                                               q8_pack4(qv[16 * c + 4], qv[16 * c + 5], qv[16 * c + 6], qv[16 * c + 7], rqw),
                                               q8_pack4(qv[16 * c + 8], qv[16 * c + 9], qv[16 * c + 10], qv[16 * c + 11], rqw),
                                               q8_pack4(qv[16 * c + 12], qv[16 * c + 13], qv[16 * c + 14], qv[16 * c + 15], rqw));
                    if (kNT == 2) {
                        *reinterpret_cast<uint4*>(sub + lane * 64 + ((cc ^ ((lane >> 1) & 3)) << 4)) = v;
                    } else if (row_valid) {
                        *reinterpret_cast<uint4*>(((half == 0) ? p.Wq : p.Uq) + grow * kD + h * kFW + cc * 16) = v;
                    }
                }
            }
            if (half == 0) {
                tc_fence_before_sync();
                cta_barrier();  // every row of the W accumulator has been read
                if (tid == 0) {
                    if (!wait_bar(&bar_v, par_kv)) {
                        ok = false;
                        *reinterpret_cast<volatile int*>(&s_fail) = 1;
                    }
                    if (ok) {
                        tc_fence_after_sync();
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const uint64_t bd = smem_desc(sV_a + ks * 4096, 16384, 1024, SWZ_128B);
                            mma_i8_ts(tmem + kR0, tmem + kAS + ks * 8, bd, idesc_m, ks > 0);
                        }
                        mma_commit(&bar_mma);
                    }
                }
            }
            if (kNT == 2) {
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_3d((half == 0) ? &tmW : &tmU, sub, h * 64, tc.t0 + wrow0, tc.bhv);
                    tma_store_commit();
                }
            }
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

// ---------------------------------------------------------------------------------------------------------------
// Chunks of 128 tokens, second kernel: the lower-left block of T and rows 64..127 of W and U (block formula of
// App. E, Eq. 28, with this path's sign: T21 = -T22 A21 T11; the stored blocks hold Abar = -A, so T21 = T22 Abar21 T11).
// The first kernel has treated the two 64-blocks of every chunk as chunks of their own (diagonal blocks of Toffq with
// their exponents, rows 0..63 of W and U are final). Here, per chunk (one tile of 128 tokens, rows 64..127 do the
// work: TMEM lanes 64..127):
//
//   G = Kq Kq^T (rows 64..127 x columns 0..63 used)                                   MMA
//   A21q = Q8(-(G o c), 2 k_exp - 15) on the full 64 x 64 block                        integer ALU
//   X    = Q8(align(A21q, A21q Toff11q));  T21q = Q8(align(X, Toff22q X))              MMA + ALU each
//   T21b = Q8(T21q_ij beta_q_j), T22b = Q8(Toff22q_ij beta_q_j)                        integer ALU
//   rows 64..127 of W: Q8(align(T21b Kq_top, T22b Kq_bot, beta_q_i Kq_i)), U likewise   two MMAs (two accumulators) + ALU
//
// One CTA per SM (512 TMEM columns: two accumulators of 128 columns and two A operands).
constexpr int kMThreads = 256;  // two threads per tile row, 32 columns of a 64-wide block each
constexpr int kMHC = 32;
__device__ __forceinline__ void mrg_barrier() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
constexpr uint32_t kMD1 = 0, kMD2 = 128, kMA1 = 256, kMA2 = 288, kMrgTmemCols = 512;
constexpr int kMOffK = 0, kMOffV = 16384, kMOffEB = 32768, kMOffBeta = 40960, kMOffDecay = kMOffBeta + 512;
constexpr int kMOffLut = kMOffDecay + 512, kMOffRed = kMOffLut + 512, kMrgSmemTotal = kMOffRed + 128;

__global__ void __launch_bounds__(kMThreads, 1)
int8_merge128_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                     const __grid_constant__ ParamsI8 p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sK = smem + kMOffK;
    uint8_t* sV = smem + kMOffV;
    uint8_t* sEB = smem + kMOffEB;
    int* sbeta = reinterpret_cast<int*>(smem + kMOffBeta);
    int* sdecay = reinterpret_cast<int*>(smem + kMOffDecay);
    uint16_t* slut = reinterpret_cast<uint16_t*>(smem + kMOffLut);
    uint32_t* sred = reinterpret_cast<uint32_t*>(smem + kMOffRed);

    __shared__ uint64_t bar_k, bar_v, bar_mma;
    __shared__ uint32_t tmem_base_s;
    __shared__ int s_fail;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    if (tid == 0) {
        mbar_init(&bar_k, 1);
        mbar_init(&bar_v, 1);
        mbar_init(&bar_mma, 1);
        s_fail = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
    }
    slut[tid] = p.lut[tid];
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, kMrgTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_s;

    const uint32_t n_tiles = static_cast<uint32_t>(p.n_tiles);
    const int n128 = p.T / kTile;
    const int t = tid & 127;        // tile row = token of the chunk
    const int h = tid >> 7;         // column half of a 64-wide block
    const int col0 = h * kMHC;
    const int il = t & (kC - 1);    // row inside its 64-block
    const int ci = t >> 6;          // 0: rows of the first block, 1: rows of the second block (the workers)
    const bool worker = ci == 1;
    const int wq = warp & 3;
    const uint32_t lane_base = tmem + (static_cast<uint32_t>(wq * 32) << 16);
    const uint32_t sK_a = smem_u32(sK), sV_a = smem_u32(sV), sEB_a = smem_u32(sEB);
    const uint32_t idesc_g = instr_desc(128, 128, 1, 1, 0, 0, 2);   // both K-major
    const uint32_t idesc_b = instr_desc(128, 64, 1, 1, 0, 1, 2);    // B MN-major, N = 64
    const uint32_t idesc_m = instr_desc(128, 128, 1, 1, 0, 1, 2);   // B MN-major, N = 128
    uint32_t par_mma = 0, par_kv = 0;

    auto failed = [&]() -> bool { return *reinterpret_cast<volatile int*>(&s_fail) != 0; };
    auto set_fail = [&]() { *reinterpret_cast<volatile int*>(&s_fail) = 1; };
    auto wait_mma = [&]() -> bool {
        if (warp == 0 && (failed() || !wait_bar(&bar_mma, par_mma))) set_fail();
        asm volatile("bar.sync 2, 256;" ::: "memory");
        par_mma ^= 1;
        return !failed();
    };
    // bit length of the OR of the workers' magnitudes (the one chunk of the tile); `slot` is fresh per use
    auto block_bitlen = [&](unsigned long long m, int slot) -> int {
        const uint32_t lo = __reduce_or_sync(0xFFFFFFFFu, static_cast<uint32_t>(m));
        const uint32_t hi = __reduce_or_sync(0xFFFFFFFFu, static_cast<uint32_t>(m >> 32));
        if (lane == 0) {
            if (lo) atomicOr(&sred[slot * 2 + 0], lo);
            if (hi) atomicOr(&sred[slot * 2 + 1], hi);
        }
        mrg_barrier();
        const unsigned long long all = (static_cast<unsigned long long>(sred[slot * 2 + 1]) << 32) | sred[slot * 2 + 0];
        return all ? 64 - __clzll(static_cast<long long>(all)) : 0;
    };
    // this thread's 32 columns of a row as a piece pair of the B operand [64 x 64] (MN-major, no swizzle): 16 columns of
    // row k per 16-byte piece, pieces of one column group 1024 bytes apart
    auto store_b_row = [&](int k, const uint32_t (&w)[8]) {
#pragma unroll
        for (int c = 0; c < 2; ++c)
            *reinterpret_cast<uint4*>(sEB + ((col0 >> 4) + c) * (16 * kC) + k * 16) =
                make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
    };
    // D1 = A1 B with A1 = 64 bytes per row in TMEM, B the [64 x 64] operand above
    auto issue_block_product = [&]() {
#pragma unroll
        for (int ks = 0; ks < kC / 32; ++ks) {
            const uint64_t bd = smem_desc(sEB_a + ks * 512, 128, 16 * kC, SWZ_NONE);
            mma_i8_ts(tmem + kMD1, tmem + kMA1 + ks * 8, bd, idesc_b, ks > 0);
        }
        mma_commit(&bar_mma);
    };

    for (uint32_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const TileCoord tc = decode_tile(tile, p);
        const int c128 = tc.t0 / kTile;
        const long long chunk = (long long)tc.bhv * n128 + c128;
        const long long grow = (long long)tc.bhv * p.T + tc.t0 + t;

        tc_fence_before_sync();
        mrg_barrier();  // the previous tile is finished with the shared arrays and the accumulators
        if (tid == 0) {
            mbar_arrive_expect_tx(&bar_k, 16384);
            tma_load_3d(sK, &tmK, &bar_k, 0, tc.t0, tc.bhk);
            mbar_arrive_expect_tx(&bar_v, 16384);
            tma_load_3d(sV, &tmV, &bar_v, 0, tc.t0, tc.bhv);
        }
        const int bq = static_cast<int>(static_cast<uint16_t>(p.beta_q[grow]));
        const int dq = p.decay_q[grow];
        const int kexp = p.k_exp[(long long)tc.bhk * n128 + c128];
        const int vexp = p.v_exp[chunk];
        const int e11 = p.t_exp[chunk * 3 + 0], e22 = p.t_exp[chunk * 3 + 2];
        // this row's 32 columns of its own diagonal block of Toffq (written by the first kernel)
        uint32_t tw[8];
        {
            const uint4* src = reinterpret_cast<const uint4*>(p.Toff + (chunk * kTile + t) * kTile + ci * kC + col0);
            const uint4 v0 = src[0], v1 = src[1];
            tw[0] = v0.x; tw[1] = v0.y; tw[2] = v0.z; tw[3] = v0.w;
            tw[4] = v1.x; tw[5] = v1.y; tw[6] = v1.z; tw[7] = v1.w;
        }
        if (h == 0) {
            sbeta[t] = bq;
            sdecay[t] = dq;
        }
        if (tid < 32) sred[tid] = 0u;
        if (tid == 0) {
            if (!wait_bar(&bar_k, par_kv)) set_fail();
            if (!failed()) {
                tc_fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const uint64_t d = smem_desc(sK_a + ks * 32, 16, 1024, SWZ_128B);
                    mma_i8_ss(tmem + kMD1, d, d, idesc_g, ks > 0);
                }
                mma_commit(&bar_mma);
            }
        }
        mrg_barrier();
        if (!wait_mma()) break;
        tc_fence_after_sync();
        int slot = 0;

        // ---- A21q = Q8(-(G o c)) on the full block (rows of the second block, columns of the first)
        int a21[kMHC];
        int eA21;
        {
            uint32_t g[kMHC];
            int cq[kMHC];
            uint32_t mlo = 0, mhi = 0;
            if (worker) {
                tmem_ld32(lane_base + kMD1 + col0, g);
                tmem_wait_ld();
#pragma unroll
                for (int jl = 0; jl < kMHC; ++jl) {
                    const int dlt = dq - sdecay[col0 + jl];
                    const int sh = dlt >> 8;
                    const int gam = (sh >= 0 && sh < 16) ? (static_cast<int>(slut[dlt & 255]) >> sh) : 0;
                    const int c = (bq * gam + (1 << 14)) >> 15;
                    cq[jl] = c;
                    const uint32_t ag = static_cast<uint32_t>(abs(static_cast<int>(g[jl])));
                    mlo |= ag * static_cast<uint32_t>(c);
                    mhi |= __umulhi(ag, static_cast<uint32_t>(c));
                }
            }
            const int r = q8_shift(block_bitlen((static_cast<unsigned long long>(mhi) << 32) | mlo, slot++));
            const uint32_t half = (1u << r) >> 1;
#pragma unroll
            for (int jl = 0; jl < kMHC; ++jl) a21[jl] = 0;
            if (worker) {
                // |G| c needs up to 36 bits: (hi, lo) pair, the rounded shift (r < 32) is one funnel shift; Aq = -G c
#pragma unroll
                for (int jl = 0; jl < kMHC; ++jl) {
                    const int gv = static_cast<int>(g[jl]);
                    const uint32_t ag = static_cast<uint32_t>(abs(gv)), c = static_cast<uint32_t>(cq[jl]);
                    const uint32_t lo = ag * c, lo2 = lo + half;
                    const uint32_t hi2 = __umulhi(ag, c) + (lo2 < lo ? 1u : 0u);
                    const int q = static_cast<int>(min(__funnelshift_r(lo2, hi2, r), 127u));
                    a21[jl] = (gv < 0) ? q : -q;
                }
            }
            eA21 = 2 * kexp - 15 + r;
        }
        // ---- X = Q8(align(A21q, A21q Toff11q)): A operand = rows of A21q, B operand = Toff11q (rows of the first block)
        {
            uint32_t w[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) w[i] = worker ? pack4(a21[4 * i], a21[4 * i + 1], a21[4 * i + 2], a21[4 * i + 3]) : 0u;
            tmem_st8(lane_base + kMA1 + h * 8, w);
            if (!worker) store_b_row(il, tw);
            fence_proxy_async_smem();
            tmem_wait_st();
            tc_fence_before_sync();
            mrg_barrier();
            if (tid == 0) {
                tc_fence_after_sync();
                issue_block_product();
            }
        }
        if (!wait_mma()) break;
        tc_fence_after_sync();
        int x[kMHC];
        int eX;
        {
            const int eref = align_ref2(eA21, eA21 + e11);
            const int sa = eA21 - eref, sp = eA21 + e11 - eref;
            int acc[kMHC];
            MaxMag mm;
            if (worker) {
                uint32_t d[kMHC];
                tmem_ld32(lane_base + kMD1 + col0, d);
                tmem_wait_ld();
#pragma unroll
                for (int jl = 0; jl < kMHC; ++jl) acc[jl] = term32(a21[jl], sa) + term32(static_cast<int>(d[jl]), sp);
#pragma unroll
                for (int jl = 0; jl < kMHC; jl += 2) mm.add2(acc[jl], acc[jl + 1]);
            }
            const int r = q8_shift(block_bitlen(mm.mag(), slot++));
#pragma unroll
            for (int jl = 0; jl < kMHC; ++jl) x[jl] = worker ? q8_32(acc[jl], r) : 0;
            eX = eref + r;
        }
        // ---- T21q = Q8(align(X, Toff22q X)): A operand = rows of Toff22q, B operand = X (rows of the second block)
        {
            if (worker) {
                uint32_t w[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) w[i] = pack4(x[4 * i], x[4 * i + 1], x[4 * i + 2], x[4 * i + 3]);
                store_b_row(il, w);
                tmem_st8(lane_base + kMA1 + h * 8, tw);
            }
            fence_proxy_async_smem();
            tmem_wait_st();
            tc_fence_before_sync();
            mrg_barrier();
            if (tid == 0) {
                tc_fence_after_sync();
                issue_block_product();
            }
        }
        if (!wait_mma()) break;
        tc_fence_after_sync();
        int t21[kMHC];
        int e21;
        {
            const int eref = align_ref2(eX, e22 + eX);
            const int s0 = eX - eref, s1 = e22 + eX - eref;
            int acc[kMHC];
            MaxMag mm;
            if (worker) {
                uint32_t d[kMHC];
                tmem_ld32(lane_base + kMD1 + col0, d);
                tmem_wait_ld();
#pragma unroll
                for (int jl = 0; jl < kMHC; ++jl) acc[jl] = term32(x[jl], s0) + term32(static_cast<int>(d[jl]), s1);
#pragma unroll
                for (int jl = 0; jl < kMHC; jl += 2) mm.add2(acc[jl], acc[jl + 1]);
            }
            const int r = q8_shift(block_bitlen(mm.mag(), slot++));
#pragma unroll
            for (int jl = 0; jl < kMHC; ++jl) t21[jl] = worker ? q8_32(acc[jl], r) : 0;
            e21 = eref + r;
        }
        // the lower-left block of Toffq (rows 64..127) and zeros in the upper-right one (rows 0..63)
        {
            uint4* dst = reinterpret_cast<uint4*>(p.Toff + (chunk * kTile + t) * kTile + (worker ? 0 : kC) + col0);
#pragma unroll
            for (int c = 0; c < 2; ++c)
                dst[c] = make_uint4(pack4(t21[16 * c + 0], t21[16 * c + 1], t21[16 * c + 2], t21[16 * c + 3]),
                                    pack4(t21[16 * c + 4], t21[16 * c + 5], t21[16 * c + 6], t21[16 * c + 7]),
                                    pack4(t21[16 * c + 8], t21[16 * c + 9], t21[16 * c + 10], t21[16 * c + 11]),
                                    pack4(t21[16 * c + 12], t21[16 * c + 13], t21[16 * c + 14], t21[16 * c + 15]));
            if (worker && il == 0 && h == 0) p.t_exp[chunk * 3 + 1] = e21;
        }
        // ---- T21b = Q8(T21q_ij beta_q_j) (columns of the first block), T22b = Q8(Toff22q_ij beta_q_j) (second block)
        int e21b, e22b;
        {
            int acc1[kMHC], acc2[kMHC];
            MaxMag m1, m2;
            if (worker) {
#pragma unroll
                for (int jl = 0; jl < kMHC; ++jl) {
                    acc1[jl] = t21[jl] * sbeta[col0 + jl];
                    acc2[jl] = byte_at(tw[jl >> 2], jl & 3) * sbeta[kC + col0 + jl];
                }
#pragma unroll
                for (int jl = 0; jl < kMHC; jl += 2) {
                    m1.add2(acc1[jl], acc1[jl + 1]);
                    m2.add2(acc2[jl], acc2[jl + 1]);
                }
            }
            const int r1 = q8_shift(block_bitlen(m1.mag(), slot++));
            const int r2 = q8_shift(block_bitlen(m2.mag(), slot++));
            e21b = e21 - 15 + r1;
            e22b = e22 - 15 + r2;
            // A1 = [T21b | 0], A2 = [0 | T22b]: 128 bytes per row (the contraction runs over the 128 tokens of the tile)
            uint32_t w1[8], w2[8], z[8];
            const Rnd q1 = make_rnd(r1), q2 = make_rnd(r2);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                z[i] = 0u;
                w1[i] = worker ? q8_pack4(acc1[4 * i], acc1[4 * i + 1], acc1[4 * i + 2], acc1[4 * i + 3], q1) : 0u;
                w2[i] = worker ? q8_pack4(acc2[4 * i], acc2[4 * i + 1], acc2[4 * i + 2], acc2[4 * i + 3], q2) : 0u;
            }
            tmem_st8(lane_base + kMA1 + h * 8, w1);
            tmem_st8(lane_base + kMA1 + 16 + h * 8, z);
            tmem_st8(lane_base + kMA2 + h * 8, z);
            tmem_st8(lane_base + kMA2 + 16 + h * 8, w2);
            tmem_wait_st();
        }
        // ---- rows 64..127 of W, then of U
        bool bad = false;
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
            const int xexp = (half == 0) ? kexp : vexp;
            const uint8_t* xtile = (half == 0) ? sK : sV;
            const uint32_t xt_a = (half == 0) ? sK_a : sV_a;
            tc_fence_before_sync();
            mrg_barrier();  // operands in place (half 0); the accumulators of W have been read (half 1)
            if (tid == 0) {
                if (half == 1 && !wait_bar(&bar_v, par_kv)) set_fail();
                if (!failed()) {
                    tc_fence_after_sync();
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        const uint64_t bd = smem_desc(xt_a + ks * 4096, 16384, 1024, SWZ_128B);
                        mma_i8_ts(tmem + kMD1, tmem + kMA1 + ks * 8, bd, idesc_m, ks > 0);
                    }
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        const uint64_t bd = smem_desc(xt_a + ks * 4096, 16384, 1024, SWZ_128B);
                        mma_i8_ts(tmem + kMD2, tmem + kMA2 + ks * 8, bd, idesc_m, ks > 0);
                    }
                    mma_commit(&bar_mma);
                }
            }
            if (!wait_mma()) { bad = true; break; }
            tc_fence_after_sync();
            const int ep1 = e21b + xexp, ep2 = e22b + xexp, ed = xexp - 15;
            const int emin = min(ep1, min(ep2, ed)), emax = max(ep1, max(ep2, ed));
            const int eref = max(emin, emax - kAlignWindow);
            const int s1 = ep1 - eref, s2 = ep2 - eref, sd = ed - eref;
            // |T b X| <= 64 * 127^2 < 2^20, |beta_q X| < 2^22; a left shift is at most 8: the sum fits 32 bits
            int sums[64];
            MaxMag mm;
            if (worker) {
                uint32_t xr[16];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint4 v = *reinterpret_cast<const uint4*>(xtile + t * 128 + (((h * 4 + c) ^ (t & 7)) << 4));
                    xr[4 * c + 0] = v.x; xr[4 * c + 1] = v.y; xr[4 * c + 2] = v.z; xr[4 * c + 3] = v.w;
                }
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t d1[32], d2[32];
                    tmem_ld32(lane_base + kMD1 + h * 64 + c0, d1);
                    tmem_ld32(lane_base + kMD2 + h * 64 + c0, d2);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        sums[c0 + i] = term32(static_cast<int>(d1[i]), s1) + term32(static_cast<int>(d2[i]), s2) +
                                       term32(bq * byte_at(xr[(c0 + i) >> 2], (c0 + i) & 3), sd);
#pragma unroll
                    for (int i = 0; i < 32; i += 2) mm.add2(sums[c0 + i], sums[c0 + i + 1]);
                }
            }
            const int rr = q8_shift(block_bitlen(mm.mag(), slot++));
            if (worker) {
                const Rnd rq = make_rnd(rr);
                if (il == 0 && h == 0) ((half == 0) ? p.w_exp : p.u_exp)[chunk * 2 + 1] = eref + rr;
                uint4* dst = reinterpret_cast<uint4*>(((half == 0) ? p.Wq : p.Uq) + grow * kD + h * 64);
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    dst[c] = make_uint4(q8_pack4(sums[16 * c + 0], sums[16 * c + 1], sums[16 * c + 2], sums[16 * c + 3], rq),
                                        q8_pack4(sums[16 * c + 4], sums[16 * c + 5], sums[16 * c + 6], sums[16 * c + 7], rq),
                                        q8_pack4(sums[16 * c + 8], sums[16 * c + 9], sums[16 * c + 10], sums[16 * c + 11], rq),
                                        q8_pack4(sums[16 * c + 12], sums[16 * c + 13], sums[16 * c + 14], sums[16 * c + 15], rq));
            }
        }
        if (bad) break;
        par_kv ^= 1;
    }
    if (failed() && tid == 0) atomicExch(p.status, GDN_ERR_TIMEOUT);

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, kMrgTmemCols);
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

// [heads][T][cols] int8 tensor
bool make_map(CUtensorMap* tm, const void* base, long long heads, int T, int cols, int box_cols, int box_rows,
              CUtensorMapSwizzle swizzle) {
    EncodeTiledFn enc = get_encode_fn();
    if (enc == nullptr) return false;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(T), static_cast<cuuint64_t>(heads)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(T) * cols};
    cuuint32_t box[3] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(box_rows), 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace


void int8_decay_lut(uint16_t* out) {
    for (int f = 0; f < 256; ++f) out[f] = static_cast<uint16_t>(floor(32768.0 * exp2(-static_cast<double>(f) / 256.0) + 0.5));
}

int launch_tc_int8(const ProblemI8& q, cudaStream_t stream) {
    if (q.d_k != kD || q.d_v != kD) return GDN_ERR_UNSUPPORTED;
    const bool merge = q.C == 2 * kC;  // chunks of 128 tokens: two 64-blocks, then the block-merge kernel
    if (q.C != kC && !merge) return GDN_ERR_UNSUPPORTED;
    if (merge && (q.Toff == nullptr || q.dbg != nullptr || q.T % (2 * kC) != 0)) return GDN_ERR_UNSUPPORTED;
    if (merge && ((reinterpret_cast<uintptr_t>(q.Toff) | reinterpret_cast<uintptr_t>(q.Wq) | reinterpret_cast<uintptr_t>(q.Uq)) & 15) != 0)
        return GDN_ERR_ALIGN;
    if (q.order < 1 || q.order > 3) return GDN_ERR_UNSUPPORTED;  // the paper limits the low-bit order to N <= 3
    if (q.steps > kSMax) return GDN_ERR_UNSUPPORTED;
    if ((long long)q.B * q.H_v * q.T == 0) return GDN_OK;
    int* status = device_status_word();
    if (status == nullptr) return GDN_ERR_LAUNCH;
    const long long hk = (long long)q.B * q.H_k, hv = (long long)q.B * q.H_v;
    CUtensorMap mK, mV, mW, mU, mT;
    if (!make_map(&mK, q.Kq, hk, q.T, kD, 128, 128, CU_TENSOR_MAP_SWIZZLE_128B)) return GDN_ERR_LAUNCH;
    if (!make_map(&mV, q.Vq, hv, q.T, kD, 128, 128, CU_TENSOR_MAP_SWIZZLE_128B)) return GDN_ERR_LAUNCH;
    if (!make_map(&mW, q.Wq, hv, q.T, kD, 64, 32, CU_TENSOR_MAP_SWIZZLE_64B)) return GDN_ERR_LAUNCH;
    if (!make_map(&mU, q.Uq, hv, q.T, kD, 64, 32, CU_TENSOR_MAP_SWIZZLE_64B)) return GDN_ERR_LAUNCH;
    if (!make_map(&mT, q.Toff != nullptr ? q.Toff : q.Wq, hv, q.T, q.Toff != nullptr ? q.C : kD, 64, 32, CU_TENSOR_MAP_SWIZZLE_64B))
        return GDN_ERR_LAUNCH;
    ParamsI8 prm;
    prm.beta_q = q.beta_q;
    prm.decay_q = q.decay_q;
    prm.k_exp = q.k_exp;
    prm.v_exp = q.v_exp;
    prm.w_exp = q.w_exp;
    prm.u_exp = q.u_exp;
    prm.t_exp = q.t_exp;
    prm.Toff = q.Toff;
    prm.dbg = q.dbg;
    prm.status = status;
    prm.H_k = q.H_k;
    prm.H_v = q.H_v;
    prm.T = q.T;
    prm.group = q.H_v / q.H_k;
    prm.n_tt = (q.T + kTile - 1) / kTile;
    prm.N = q.order;
    prm.S = q.steps;
    prm.merge = merge ? 1 : 0;
    prm.Wq = q.Wq;
    prm.Uq = q.Uq;
    prm.n_tiles = hv * prm.n_tt;
    if (prm.n_tiles >= (1LL << 31) - 4096) return GDN_ERR_UNSUPPORTED;
    int8_decay_lut(prm.lut);
    const int smem = kSmemTotal + 1024;
    if (cudaFuncSetAttribute(chunk_tc_int8_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
        cudaFuncSetAttribute(chunk_tc_int8_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
        return GDN_ERR_LAUNCH;
    const long long grid = prm.n_tiles < 2 * 148 ? prm.n_tiles : 2 * 148;
    if (q.dbg != nullptr) chunk_tc_int8_kernel<true><<<static_cast<int>(grid), kThreads, smem, stream>>>(mK, mV, mW, mU, mT, prm);
    else chunk_tc_int8_kernel<false><<<static_cast<int>(grid), kThreads, smem, stream>>>(mK, mV, mW, mU, mT, prm);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) return GDN_ERR_LAUNCH;
    if (merge) {
        const int smem2 = kMrgSmemTotal + 1024;
        if (cudaFuncSetAttribute(int8_merge128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem2) != cudaSuccess)
            return GDN_ERR_LAUNCH;
        const long long grid2 = prm.n_tiles < 148 ? prm.n_tiles : 148;
        int8_merge128_kernel<<<static_cast<int>(grid2), kMThreads, smem2, stream>>>(mK, mV, prm);
        count_launch();
    }
    return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_LAUNCH;
}

}  // namespace gdn
