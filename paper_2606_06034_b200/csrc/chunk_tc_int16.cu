// INT16 variant of the chunk-prepare path (the paper's primary integer precision for the inverse: Sec. 4.2, Table 1;
// App. G table, row "Matrix Inversion") on the tensor cores.
//
// Every tensor of the chain is int16 mantissas in [-32767, 32767] with one power-of-two exponent per chunk; the steps
// are those of the INT8 kernel with Q16 in place of Q8 (uniform symmetric quantiser of App. G, Eq. 32; N <= 3 with
// residual correction, Sec. 3.5; band mask before every requantisation, Sec. 3.3):
//
//   rsr(x, r)   = sign(x) ((|x| + 2^(r-1)) >> r)
//   Q16(acc, e) : r = max(0, bitlen(max |acc| on the support) - 15); q = clamp(rsr(acc, r), +-32767); exponent e + r
//   align(..)   : e_ref = max(min e, max e - 16); terms shifted to e_ref (left shift, or rsr) and summed in 64 bits
//
// B200 has no 16-bit integer tensor path, so every matrix product runs on tcgen05 kind::i8 over BYTE PLANES: a mantissa
// x = 256 xh + xl with xh = x >> 8 (signed byte) and xl = x & 255 (unsigned byte), and
//   X Y = 65536 Xh Yh + 256 (Xh Yl + Xl Yh) + Xl Yl,
// four products with the operand types (s8,s8), (s8,u8), (u8,s8), (u8,u8) into three int32 accumulators in TMEM (the two
// mixed ones share one); the threads recombine them exactly in 64 bits. The K and V tiles arrive as int16 by TMA and are
// split into byte planes in shared memory by the threads.
//
// One CTA of 256 threads per SM (three 128-column accumulators + two operand planes = 448 TMEM columns), tile of 128
// tokens = two 64-chunks, threads t and t + 128 share tile row t and split its 64 chunk columns. Everything between the
// products is 64-bit integer ALU work; the kernel is written for exactness, not tuned.
#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace gdn {
namespace {

using namespace sm100;

constexpr int kTile = 128;
constexpr int kThreads = 256;
constexpr int kD = 128;
constexpr int kC = 64;
constexpr int kHC = 32;          // chunk columns per thread
constexpr int kSMax = 8;
constexpr int kWin = 16;         // bits kept below the largest term of an aligned sum
constexpr int kQ = 32767;
// TMEM columns: three accumulators (hi*hi, mixed, lo*lo) and the two byte planes of the A operand
constexpr uint32_t kDhh = 0, kDmid = 128, kDll = 256, kAh = 384, kAl = 416, kTmemCols = 512;

struct ParamsI16 {
    const int16_t* beta_q;
    const int32_t* decay_q;
    const int32_t* k_exp;
    const int32_t* v_exp;
    int16_t* W;
    int16_t* U;
    int32_t* w_exp;
    int32_t* u_exp;
    int32_t* t_exp;
    int16_t* Toff;   // may be null
    long long* dbg;  // may be null: [heads * chunks][64][8 * 64 + 128 + 128] exact matrix products
    int* status;
    int H_k, H_v, T, group, n_tt;
    int N, S;
    long long n_tiles;
    uint16_t lut[256];
};

// shared memory map (bytes)
constexpr int kOffK16 = 0;                 // 32 KB: int16 K tile, two [128][64] boxes, 128-byte swizzle
constexpr int kOffV16 = 32768;             // 32 KB
constexpr int kOffPh = 65536;              // 16 KB: high-byte plane of K (then V), [128][128] bytes, 128-byte swizzle
constexpr int kOffPl = kOffPh + 16384;     // 16 KB: low-byte plane
constexpr int kOffEh = kOffPl + 16384;     // 8 KB: high bytes of Eq as B operand [64 x 128] (MN-major, no swizzle)
constexpr int kOffEl = kOffEh + 8192;      // 8 KB
constexpr int kOffRow = kOffEl + 8192;     // 16 KB: one private row of 64 int16 per tile row (Aq, later Sq)
constexpr int kOffSH = kOffRow + 16384;    // column form of T0q: [128 + 8][4] int
constexpr int kOffAB = kOffSH + 136 * 16;  // row form: band of Aq / P_2: [128][8] int
constexpr int kOffBeta = kOffAB + 128 * 32;
constexpr int kOffDecay = kOffBeta + 512;
constexpr int kOffLut = kOffDecay + 512;
constexpr int kOffRed = kOffLut + 512;     // OR-reduction slots: [24][2 chunks][2 words]
constexpr int kNumRed = 24;
constexpr int kOffPark = (kOffRed + kNumRed * 16 + 1023) / 1024 * 1024;  // 80 KB: parked rows of R_4..R_8 (see the kernel)
constexpr int kSmemTotal = kOffPark + 5 * 16384;

__device__ __forceinline__ void cta_barrier() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t i = 0;
    while (!mbar_try_wait_hint(bar, parity, 2000u)) {
        if ((++i & 63u) == 0 && clock64() - t0 > 2000000000LL) return false;
    }
    return true;
}

// rounded right shift, half away from zero (0 <= r <= 62), without branches: for x < 0 the rounded shift of the
// magnitude equals the arithmetic shift of x + half - 1 (floor((x + h - 1) / 2^r) = -floor((|x| + h) / 2^r) because
// 2^r - h = h); r = 0 gives x. r is uniform over a chunk, so the constants are computed once per stage.
__device__ __forceinline__ long long rsr64(long long x, int r) {
    const long long half = static_cast<long long>((1ull << r) >> 1);
    const long long neg1 = (r > 0) ? (x >> 63) : 0;
    return (x + half + neg1) >> r;
}
// one term of an aligned sum: x 2^s for s >= 0, rounded right shift otherwise
__device__ __forceinline__ long long term64(long long x, int s) {
    const int r = s >= 0 ? 0 : ((-s) < 62 ? (-s) : 62);
    return rsr64(x, r) << (s >= 0 ? s : 0);
}
// clamp(rsr(x, r), +-kQ). r is the shift of the chunk's largest magnitude (q_shift of its bit length), so the shifted
// value is at most 2^15 in magnitude and the clamp is done in 32 bits.
__device__ __forceinline__ int q16(long long x, int r) {
    const int y = static_cast<int>(rsr64(x, r));
    return max(min(y, kQ), -kQ);
}
__device__ __forceinline__ unsigned long long abs64(long long x) { return static_cast<unsigned long long>(x < 0 ? -x : x); }
__device__ __forceinline__ int q_shift(int bitlen) { return bitlen > 15 ? bitlen - 15 : 0; }
__device__ __forceinline__ int align_ref2(int e0, int e1) {
    const int lo = e0 < e1 ? e0 : e1, hi = e0 < e1 ? e1 : e0;
    return lo > hi - kWin ? lo : hi - kWin;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
// two mantissas as one word of int16 pairs
__device__ __forceinline__ uint32_t pack2(int a, int b) { return prmt(static_cast<uint32_t>(a), static_cast<uint32_t>(b), 0x5410u); }
__device__ __forceinline__ int lo16(uint32_t w) { return static_cast<int>(static_cast<int16_t>(w & 0xFFFFu)); }
__device__ __forceinline__ int hi16(uint32_t w) { return static_cast<int>(w) >> 16; }
// byte planes of four mantissas held as two int16-pair words: low bytes / high bytes, element order kept
__device__ __forceinline__ uint32_t plane_lo(uint32_t w0, uint32_t w1) { return prmt(w0, w1, 0x6420u); }
__device__ __forceinline__ uint32_t plane_hi(uint32_t w0, uint32_t w1) { return prmt(w0, w1, 0x7531u); }
// exact product sum from the three byte-plane accumulators
__device__ __forceinline__ long long combine(uint32_t hh, uint32_t mid, uint32_t ll) {
    return (static_cast<long long>(static_cast<int>(hh)) << 16) + (static_cast<long long>(static_cast<int>(mid)) << 8) +
           static_cast<long long>(static_cast<int>(ll));
}

struct TileCoord {
    int bhk, bhv, t0;
};
__device__ __forceinline__ TileCoord decode_tile(uint32_t tile, const ParamsI16& p) {
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

// DBG: the instantiation that also writes every exact matrix product (tests of small cases); the normal one carries
// none of its tests and stores.
template <bool DBG>
__global__ void __launch_bounds__(kThreads, 1)
chunk_tc_int16_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                      const __grid_constant__ ParamsI16 p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sK16 = smem + kOffK16;
    uint8_t* sV16 = smem + kOffV16;
    uint8_t* sPh = smem + kOffPh;
    uint8_t* sPl = smem + kOffPl;
    uint8_t* sEh = smem + kOffEh;
    uint8_t* sEl = smem + kOffEl;
    uint8_t* sRow = smem + kOffRow;
    int* sSH = reinterpret_cast<int*>(smem + kOffSH);
    int* sAB = reinterpret_cast<int*>(smem + kOffAB);
    int* sbeta = reinterpret_cast<int*>(smem + kOffBeta);
    int* sdecay = reinterpret_cast<int*>(smem + kOffDecay);
    uint16_t* slut = reinterpret_cast<uint16_t*>(smem + kOffLut);
    uint32_t* sred = reinterpret_cast<uint32_t*>(smem + kOffRed);

    __shared__ uint64_t bar_k, bar_v, bar_mma;
    __shared__ uint32_t tmem_base_s;
    __shared__ int s_fail;  // set when a bounded wait ran out

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
        tmem_alloc(&tmem_base_s, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_s;

    const int N = p.N, S = p.S;
    const uint32_t n_tiles = static_cast<uint32_t>(p.n_tiles);
    const int n_c = p.T / kC;

    const int t = tid & 127;        // tile row
    const int h = tid >> 7;         // column half
    const int col0 = h * kHC;       // first chunk column of this thread
    const int il = t & (kC - 1);    // row inside the chunk
    const int cb = t - il;          // first tile row of the chunk
    const int ci = t >> 6;          // chunk of the tile
    const int wq = warp & 3;
    const uint32_t lane_base = tmem + (static_cast<uint32_t>(wq * 32) << 16);
    const uint32_t sPh_a = smem_u32(sPh), sPl_a = smem_u32(sPl), sEh_a = smem_u32(sEh), sEl_a = smem_u32(sEl);
    // operand types of the four byte-plane products (0 = u8, 1 = s8); B K-major for the Gram matrix, MN-major otherwise
    const uint32_t idg_ss = instr_desc(128, 128, 1, 1, 0, 0, 2), idg_su = instr_desc(128, 128, 1, 0, 0, 0, 2);
    const uint32_t idg_us = instr_desc(128, 128, 0, 1, 0, 0, 2), idg_uu = instr_desc(128, 128, 0, 0, 0, 0, 2);
    const uint32_t idm_ss = instr_desc(128, 128, 1, 1, 0, 1, 2), idm_su = instr_desc(128, 128, 1, 0, 0, 1, 2);
    const uint32_t idm_us = instr_desc(128, 128, 0, 1, 0, 1, 2), idm_uu = instr_desc(128, 128, 0, 0, 0, 1, 2);
    uint32_t par_mma = 0, par_kv = 0;

    auto failed = [&]() -> bool { return *reinterpret_cast<volatile int*>(&s_fail) != 0; };
    auto set_fail = [&]() { *reinterpret_cast<volatile int*>(&s_fail) = 1; };
    // completion of the products committed to bar_mma: warp 0 polls, the others sleep on a hardware barrier; a wait that
    // ran out is published in s_fail so that all threads leave the tile loop at the same point
    auto wait_mma = [&]() -> bool {
        if (warp == 0 && (failed() || !wait_bar(&bar_mma, par_mma))) set_fail();
        asm volatile("bar.sync 2, 256;" ::: "memory");
        par_mma ^= 1;
        return !failed();
    };
    // bit length of the OR of |values| over the chunk; `slot` is a fresh reduction slot of this tile
    auto chunk_bitlen = [&](unsigned long long m, int slot) -> int {
        const uint32_t lo = __reduce_or_sync(0xFFFFFFFFu, static_cast<uint32_t>(m));
        const uint32_t hi = __reduce_or_sync(0xFFFFFFFFu, static_cast<uint32_t>(m >> 32));
        if (lane == 0) {
            if (lo) atomicOr(&sred[(slot * 2 + ci) * 2 + 0], lo);
            if (hi) atomicOr(&sred[(slot * 2 + ci) * 2 + 1], hi);
        }
        cta_barrier();
        const unsigned long long all =
            (static_cast<unsigned long long>(sred[(slot * 2 + ci) * 2 + 1]) << 32) | sred[(slot * 2 + ci) * 2 + 0];
        return all ? 64 - __clzll(static_cast<long long>(all)) : 0;
    };
    // this thread's 64 int16 of its row of an int16 tile (columns [64 h, 64 h + 64)) as 32 words
    auto load_row16 = [&](const uint8_t* tile16, uint32_t (&w)[32]) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint4 v = *reinterpret_cast<const uint4*>(tile16 + h * 16384 + t * 128 + ((c ^ (t & 7)) << 4));
            w[4 * c + 0] = v.x; w[4 * c + 1] = v.y; w[4 * c + 2] = v.z; w[4 * c + 3] = v.w;
        }
    };
    // int16 tile -> byte planes (K-major, 128-byte swizzle): this thread's 64 elements are bytes [64 h, 64 h + 64) of row t
    auto split_planes = [&](const uint8_t* tile16) {
        uint32_t w[32];
        load_row16(tile16, w);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint4 lo = make_uint4(plane_lo(w[8 * c + 0], w[8 * c + 1]), plane_lo(w[8 * c + 2], w[8 * c + 3]),
                                        plane_lo(w[8 * c + 4], w[8 * c + 5]), plane_lo(w[8 * c + 6], w[8 * c + 7]));
            const uint4 hi = make_uint4(plane_hi(w[8 * c + 0], w[8 * c + 1]), plane_hi(w[8 * c + 2], w[8 * c + 3]),
                                        plane_hi(w[8 * c + 4], w[8 * c + 5]), plane_hi(w[8 * c + 6], w[8 * c + 7]));
            const int pos = ((h * 4 + c) ^ (t & 7)) << 4;
            *reinterpret_cast<uint4*>(sPl + t * 128 + pos) = lo;
            *reinterpret_cast<uint4*>(sPh + t * 128 + pos) = hi;
        }
    };
    // the four byte-plane products of one matrix product, issued by one thread: A planes in TMEM (n_ks steps of 32
    // bytes, 8 columns each), B planes in shared memory (descriptor of step ks from bdesc)
    auto issue_ts = [&](int n_ks, uint32_t bh_a, uint32_t bl_a, uint32_t ks_bytes, uint32_t lbo, uint32_t sbo, uint32_t swz) {
        for (int ks = 0; ks < n_ks; ++ks)
            mma_i8_ts(tmem + kDhh, tmem + kAh + ks * 8, smem_desc(bh_a + ks * ks_bytes, lbo, sbo, swz), idm_ss, ks > 0);
        for (int ks = 0; ks < n_ks; ++ks)
            mma_i8_ts(tmem + kDmid, tmem + kAh + ks * 8, smem_desc(bl_a + ks * ks_bytes, lbo, sbo, swz), idm_su, ks > 0);
        for (int ks = 0; ks < n_ks; ++ks)
            mma_i8_ts(tmem + kDmid, tmem + kAl + ks * 8, smem_desc(bh_a + ks * ks_bytes, lbo, sbo, swz), idm_us, true);
        for (int ks = 0; ks < n_ks; ++ks)
            mma_i8_ts(tmem + kDll, tmem + kAl + ks * 8, smem_desc(bl_a + ks * ks_bytes, lbo, sbo, swz), idm_uu, ks > 0);
        mma_commit(&bar_mma);
    };

    if (tid == 0 && blockIdx.x < n_tiles) {
        const TileCoord c = decode_tile(blockIdx.x, p);
        mbar_arrive_expect_tx(&bar_k, 32768);
        tma_load_3d(sK16, &tmK, &bar_k, 0, c.t0, c.bhk);
        tma_load_3d(sK16 + 16384, &tmK, &bar_k, 64, c.t0, c.bhk);
    }

    for (uint32_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const TileCoord tc = decode_tile(tile, p);
        const uint32_t next = tile + gridDim.x;
        const bool has_next = next < n_tiles;
        const bool row_valid = (tc.t0 + t) < p.T;
        const long long grow = (long long)tc.bhv * p.T + tc.t0 + t;
        const int chunk_in_head = (tc.t0 + cb) / kC;
        const bool chunk_valid = (tc.t0 + cb) < p.T;
        const long long chunk_id = (long long)tc.bhv * n_c + chunk_in_head;
        constexpr int kDbgRow = 8 * kC + 2 * kD;
        long long* dbg_row = (DBG && p.dbg != nullptr && row_valid) ? p.dbg + (chunk_id * kC + il) * kDbgRow : nullptr;

        int bq = 0, dq = 0, kexp = 0, vexp = 0;
        if (row_valid) {
            bq = static_cast<int>(static_cast<uint16_t>(p.beta_q[grow]));
            dq = p.decay_q[grow];
        }
        if (chunk_valid) {
            kexp = p.k_exp[(long long)tc.bhk * n_c + chunk_in_head];
            vexp = p.v_exp[(long long)tc.bhv * n_c + chunk_in_head];
        }
        tc_fence_before_sync();
        cta_barrier();  // the previous tile is finished with the shared arrays, the V tile and the accumulators
        if (tid == 0) {
            if (!wait_bar(&bar_k, par_kv)) set_fail();
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
        cta_barrier();  // the K tile has arrived (or the wait failed)
        if (failed()) break;
        int slot = 0;

        // ---- byte planes of K, then G = Kq Kq^T as four byte-plane products
        split_planes(sK16);
        fence_proxy_async_smem();
        tc_fence_before_sync();
        cta_barrier();
        if (tid == 0) {
            tc_fence_after_sync();
            for (int ks = 0; ks < 4; ++ks) {
                const uint64_t dh = smem_desc(sPh_a + ks * 32, 16, 1024, SWZ_128B);
                mma_i8_ss(tmem + kDhh, dh, dh, idg_ss, ks > 0);
            }
            for (int ks = 0; ks < 4; ++ks) {
                const uint64_t dh = smem_desc(sPh_a + ks * 32, 16, 1024, SWZ_128B), dl = smem_desc(sPl_a + ks * 32, 16, 1024, SWZ_128B);
                mma_i8_ss(tmem + kDmid, dh, dl, idg_su, ks > 0);
            }
            for (int ks = 0; ks < 4; ++ks) {
                const uint64_t dh = smem_desc(sPh_a + ks * 32, 16, 1024, SWZ_128B), dl = smem_desc(sPl_a + ks * 32, 16, 1024, SWZ_128B);
                mma_i8_ss(tmem + kDmid, dl, dh, idg_us, true);
            }
            for (int ks = 0; ks < 4; ++ks) {
                const uint64_t dl = smem_desc(sPl_a + ks * 32, 16, 1024, SWZ_128B);
                mma_i8_ss(tmem + kDll, dl, dl, idg_uu, ks > 0);
            }
            mma_commit(&bar_mma);
        }
        if (!wait_mma()) break;
        tc_fence_after_sync();

        // ---- I1-I3: Aq = Q16(-(G o c))
        int aq[kHC];
        int eA;
        {
            uint32_t ghh[kHC], gmid[kHC], gll[kHC];
            tmem_ld32(lane_base + kDhh + cb + col0, ghh);
            tmem_ld32(lane_base + kDmid + cb + col0, gmid);
            tmem_ld32(lane_base + kDll + cb + col0, gll);
            tmem_wait_ld();
            long long acc[kHC];
            unsigned long long m = 0;
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) {
                const long long G = combine(ghh[jl], gmid[jl], gll[jl]);
                if (DBG && dbg_row != nullptr) dbg_row[col0 + jl] = G;
                const int j = col0 + jl;
                const int dlt = dq - sdecay[cb + j];
                const int sh = dlt >> 8;
                const int gam = (sh >= 0 && sh < 16) ? (static_cast<int>(slut[dlt & 255]) >> sh) : 0;
                const int c = (j < il) ? ((bq * gam + (1 << 14)) >> 15) : 0;
                acc[jl] = -G * static_cast<long long>(c);
                m |= abs64(acc[jl]);
            }
            const int r = q_shift(chunk_bitlen(m, slot++));
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) aq[jl] = q16(acc[jl], r);
            eA = 2 * kexp - 15 + r;
        }
        // Aq to the private row; entries next to the diagonal and right of this half come back from there
        int16_t* rowa = reinterpret_cast<int16_t*>(sRow + t * 128);
        {
#pragma unroll
            for (int c = 0; c < 4; ++c)
                *reinterpret_cast<uint4*>(sRow + t * 128 + col0 * 2 + c * 16) =
                    make_uint4(pack2(aq[8 * c + 0], aq[8 * c + 1]), pack2(aq[8 * c + 2], aq[8 * c + 3]),
                               pack2(aq[8 * c + 4], aq[8 * c + 5]), pack2(aq[8 * c + 6], aq[8 * c + 7]));
        }
        cta_barrier();
        int ab1 = 0, ab2 = 0, ab3 = 0;  // Aq[i][i-1..i-3]
        if (il >= 1) ab1 = rowa[il - 1];
        if (il >= 2) ab2 = rowa[il - 2];
        if (il >= 3) ab3 = rowa[il - 3];
        int an0 = 0, an1 = 0, an2 = 0;  // Aq[i][32..34] for the left half
        if (h == 0) {
            an0 = rowa[kHC + 0];
            an1 = rowa[kHC + 1];
            an2 = rowa[kHC + 2];
        }
        const int p11 = ab1, p12 = (N >= 2) ? ab2 : 0, p13 = (N >= 3) ? ab3 : 0;  // P_1 = band of Aq
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
            const long long acc22 = (N >= 2) ? (long long)p11 * sAB[r1 * 8 + 1] : 0;
            const long long acc23 = (N >= 3) ? (long long)p11 * sAB[r1 * 8 + 2] + (long long)p12 * sAB[r2 * 8 + 1] : 0;
            int p22 = 0, p23 = 0, p33 = 0;
            int e2 = 0, e3 = 0;
            if (N >= 2) {
                const unsigned long long m = (h == 0) ? (abs64(acc22) | abs64(acc23)) : 0ull;
                const int r = q_shift(chunk_bitlen(m, slot++));
                p22 = q16(acc22, r);
                p23 = q16(acc23, r);
                e2 = eA + eA + r;
            }
            if (N >= 3) {
                // P_3 at distance 3: P_2[i][i-2] * Aq[i-2][i-3]
                const long long acc3 = (long long)p22 * sAB[r2 * 8 + 1];
                const int r = q_shift(chunk_bitlen((h == 0) ? abs64(acc3) : 0ull, slot++));
                p33 = q16(acc3, r);
                e3 = e2 + eA + r;
            }
            int emin = eA, emax = eA;
            if (N >= 2) { emin = min(emin, e2); emax = max(emax, e2); }
            if (N >= 3) { emin = min(emin, e3); emax = max(emax, e3); }
            const int eref = max(emin, emax - kWin);
            const int s1 = eA - eref, s2 = e2 - eref, s3 = e3 - eref;
            long long a1 = term64(p11, s1);
            long long a2 = term64(p12, s1) + ((N >= 2) ? term64(p22, s2) : 0);
            long long a3 = term64(p13, s1) + ((N >= 2) ? term64(p23, s2) : 0) + ((N >= 3) ? term64(p33, s3) : 0);
            if (!(N >= 1 && il >= 1)) a1 = 0;
            if (!(N >= 2 && il >= 2)) a2 = 0;
            if (!(N >= 3 && il >= 3)) a3 = 0;
            const unsigned long long m = (h == 0) ? (abs64(a1) | abs64(a2) | abs64(a3)) : 0ull;
            const int r = q_shift(chunk_bitlen(m, slot++));
            t0q1 = q16(a1, r);
            t0q2 = q16(a2, r);
            t0q3 = q16(a3, r);
            eT0 = eref + r;
            if (h == 0) {
                if (il >= 1) sSH[(t - 1) * 4 + 0] = t0q1;
                if (il >= 2) sSH[(t - 2) * 4 + 1] = t0q2;
                if (il >= 3) sSH[(t - 3) * 4 + 2] = t0q3;
            }
            cta_barrier();
        }

        // ---- I6: Eq = Q16(align(Aq, Aq T0q)) on i-j > N
        int eq[kHC];
        int eE;
        {
            const int eref = align_ref2(eA, eA + eT0);
            const int sa = eA - eref, sp = eA + eT0 - eref;
            long long acc[kHC];
            unsigned long long m = 0;
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) {
                const int4 c4 = *reinterpret_cast<const int4*>(sSH + (cb + col0 + jl) * 4);
                const int a1 = (jl + 1 < kHC) ? aq[(jl + 1 < kHC) ? jl + 1 : 0] : ((jl + 1 == kHC) ? an0 : (jl + 1 == kHC + 1 ? an1 : an2));
                const int a2 = (jl + 2 < kHC) ? aq[(jl + 2 < kHC) ? jl + 2 : 0] : ((jl + 2 == kHC) ? an0 : (jl + 2 == kHC + 1 ? an1 : an2));
                const int a3 = (jl + 3 < kHC) ? aq[(jl + 3 < kHC) ? jl + 3 : 0] : ((jl + 3 == kHC) ? an0 : (jl + 3 == kHC + 1 ? an1 : an2));
                const bool on = (il - (col0 + jl)) > N;
                const long long pr = (long long)a1 * c4.x + (long long)a2 * c4.y + (long long)a3 * c4.z;
                const long long v = on ? (term64(aq[jl], sa) + term64(pr, sp)) : 0;
                acc[jl] = v;
                m |= abs64(v);
            }
            const int r = q_shift(chunk_bitlen(m, slot++));
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) eq[jl] = q16(acc[jl], r);
            eE = eref + r;
        }
        // Rows of the powers R_s (R_1 = Eq) as int16 pairs. The loops over the powers are NOT unrolled (the kernel is bound
        // by instruction fetch), so the rows cannot sit in registers indexed by s: every thread parks its 64 bytes of R_s
        // in shared memory and reads them back for the sum. The parked rows are private to the thread (no barrier):
        // R_1 in its private row (the Aq row there is dead), R_2 and R_3 in the V tile's buffer (V is loaded after the
        // sum), R_4..R_8 in a region of their own.
        auto park = [&](int s) -> uint8_t* {
            uint8_t* base = (s == 1) ? sRow : (s <= 3 ? sV16 + (s - 2) * 16384 : smem + kOffPark + (s - 4) * 16384);
            return base + t * 128 + h * 64;
        };
        uint32_t cur[kHC / 2];  // R_{s-1} inside the loop
        int er[kSMax];
#pragma unroll
        for (int s = 0; s < kSMax; ++s) er[s] = 0;
#pragma unroll
        for (int w = 0; w < kHC / 2; ++w) cur[w] = 0u;
        int n_terms = 0;
        if (S >= 1) {
#pragma unroll
            for (int w = 0; w < kHC / 2; ++w) cur[w] = pack2(eq[2 * w], eq[2 * w + 1]);
            er[0] = eE;
            n_terms = 1;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                *reinterpret_cast<uint4*>(park(1) + c * 16) = make_uint4(cur[4 * c], cur[4 * c + 1], cur[4 * c + 2], cur[4 * c + 3]);
            // B operand [E_1 | E_2] as two byte planes (64 x 128 bytes each, MN-major, no swizzle): 16 columns of
            // chunk-row il per 16-byte piece
#pragma unroll
            for (int c = 0; c < kHC / 16; ++c) {
                const uint32_t* w = &cur[8 * c];
                const uint32_t off = (((cb + col0) >> 4) + c) * (16 * kC) + il * 16;
                *reinterpret_cast<uint4*>(sEl + off) = make_uint4(plane_lo(w[0], w[1]), plane_lo(w[2], w[3]), plane_lo(w[4], w[5]), plane_lo(w[6], w[7]));
                *reinterpret_cast<uint4*>(sEh + off) = make_uint4(plane_hi(w[0], w[1]), plane_hi(w[2], w[3]), plane_hi(w[4], w[5]), plane_hi(w[6], w[7]));
            }
        }
        // ---- I7: R_s = Q16(R_{s-1} Eq) while s (N+1) < C
        bool bad = false;
#pragma unroll 1
        for (int s = 2; s <= kSMax; ++s) {
            if (s > S || s * (N + 1) >= kC) break;
            {
                // A operand: the rows of R_{s-1}, chunks stacked along M, as byte planes (64 bytes = 16 columns per plane)
                uint32_t lo8[8], hi8[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    lo8[i] = plane_lo(cur[2 * i], cur[2 * i + 1]);
                    hi8[i] = plane_hi(cur[2 * i], cur[2 * i + 1]);
                }
                tmem_st8(lane_base + kAh + h * 8, hi8);
                tmem_st8(lane_base + kAl + h * 8, lo8);
            }
            fence_proxy_async_smem();
            tmem_wait_st();
            tc_fence_before_sync();
            cta_barrier();
            if (tid == 0) {
                tc_fence_after_sync();
                issue_ts(kC / 32, sEh_a, sEl_a, 512, 128, 16 * kC, SWZ_NONE);
            }
            if (!wait_mma()) { bad = true; break; }
            tc_fence_after_sync();
            uint32_t dhh[kHC], dmid[kHC], dll[kHC];
            tmem_ld32(lane_base + kDhh + cb + col0, dhh);
            tmem_ld32(lane_base + kDmid + cb + col0, dmid);
            tmem_ld32(lane_base + kDll + cb + col0, dll);
            tmem_wait_ld();
            unsigned long long m = 0;
            long long acc[kHC];
            // R_{s-1} is zero for i - j < (s - 1)(N + 1) and Eq for i - j <= N: the integer product is exactly zero for
            // i - j < s (N + 1), no mask needed
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) {
                acc[jl] = combine(dhh[jl], dmid[jl], dll[jl]);
                if (DBG && dbg_row != nullptr) dbg_row[(s - 1) * kC + col0 + jl] = acc[jl];
                m |= abs64(acc[jl]);
            }
            const int r = q_shift(chunk_bitlen(m, slot++));
#pragma unroll
            for (int w = 0; w < kHC / 2; ++w) cur[w] = pack2(q16(acc[2 * w], r), q16(acc[2 * w + 1], r));
#pragma unroll
            for (int c = 0; c < 4; ++c)
                *reinterpret_cast<uint4*>(park(s) + c * 16) = make_uint4(cur[4 * c], cur[4 * c + 1], cur[4 * c + 2], cur[4 * c + 3]);
            er[s - 1] = er[s - 2] + eE + r;
            n_terms = s;
        }
        if (bad) break;

        // ---- Sq = Q16(align(R_1..)): a term whose right shift exceeds 15 rounds to zero and is skipped
        int sq[kHC];
        int eS = 0;
        if (n_terms > 0) {
            int emin = er[0], emax = er[0];
#pragma unroll
            for (int s = 1; s < kSMax; ++s)
                if (s < n_terms) { emin = min(emin, er[s]); emax = max(emax, er[s]); }
            const int eref = max(emin, emax - kWin);
            long long acc[kHC];
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) acc[jl] = 0;
#pragma unroll 1
            for (int s = 1; s <= n_terms; ++s) {
                const int sh = er[s - 1] - eref;
                if (sh < -15) continue;
                uint32_t w[kHC / 2];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint4 v = *reinterpret_cast<const uint4*>(park(s) + c * 16);
                    w[4 * c] = v.x; w[4 * c + 1] = v.y; w[4 * c + 2] = v.z; w[4 * c + 3] = v.w;
                }
                if (sh >= 0) {
#pragma unroll
                    for (int i = 0; i < kHC / 2; ++i) {
                        acc[2 * i] += static_cast<long long>(lo16(w[i])) << sh;
                        acc[2 * i + 1] += static_cast<long long>(hi16(w[i])) << sh;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < kHC / 2; ++i) {
                        acc[2 * i] += rsr64(lo16(w[i]), -sh);
                        acc[2 * i + 1] += rsr64(hi16(w[i]), -sh);
                    }
                }
            }
            unsigned long long m = 0;
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) m |= abs64(acc[jl]);
            fence_proxy_async_smem();  // the parked rows in the V buffer are overwritten by a bulk copy next
            const int r = q_shift(chunk_bitlen(m, slot++));
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) sq[jl] = q16(acc[jl], r);
            eS = eref + r;
        } else {
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) sq[jl] = 0;
        }
        // the V tile of this tile: its buffer held parked rows until the sum above (every thread is past its reads: the
        // reduction of the sum is a barrier), and the previous tile's U stage is long finished
        if (n_terms == 0) cta_barrier();
        if (tid == 0) {
            mbar_arrive_expect_tx(&bar_v, 32768);
            tma_load_3d(sV16, &tmV, &bar_v, 0, tc.t0, tc.bhv);
            tma_load_3d(sV16 + 16384, &tmV, &bar_v, 64, tc.t0, tc.bhv);
        }
        // Sq to the private rows (the rows above are needed for T0q Sq)
#pragma unroll
        for (int c = 0; c < 4; ++c)
            *reinterpret_cast<uint4*>(sRow + t * 128 + col0 * 2 + c * 16) =
                make_uint4(pack2(sq[8 * c + 0], sq[8 * c + 1]), pack2(sq[8 * c + 2], sq[8 * c + 3]),
                           pack2(sq[8 * c + 4], sq[8 * c + 5]), pack2(sq[8 * c + 6], sq[8 * c + 7]));
        cta_barrier();

        // ---- I8: Toffq = Q16(align(T0q, Sq, T0q Sq)) on i > j
        int toff[kHC];
        int eT;
        {
            long long prod[kHC];
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) prod[jl] = 0;
#pragma unroll
            for (int e = 1; e <= 3; ++e) {
                const int rr = (t - e) > 0 ? (t - e) : 0;
                const int cf = (il - e >= 0) ? (e == 1 ? t0q1 : (e == 2 ? t0q2 : t0q3)) : 0;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint4 a = *reinterpret_cast<const uint4*>(sRow + rr * 128 + col0 * 2 + c * 16);
                    const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        prod[8 * c + 2 * i] += (long long)cf * lo16(w[i]);
                        prod[8 * c + 2 * i + 1] += (long long)cf * hi16(w[i]);
                    }
                }
            }
            const int e0 = eT0, e1 = eS, e2 = eT0 + eS;
            const int emin = min(e0, min(e1, e2)), emax = max(e0, max(e1, e2));
            const int eref = max(emin, emax - kWin);
            const int s0 = e0 - eref, s1 = e1 - eref, s2 = e2 - eref;
            // the band entry and Sq never share an element (band: distance <= N, Sq: distance > N)
            long long acc[kHC];
            unsigned long long m = 0;
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) {
                const int d = il - (col0 + jl);
                int v = sq[jl];
                if (d == 1 && N >= 1) v = t0q1;
                if (d == 2 && N >= 2) v = t0q2;
                if (d == 3 && N >= 3) v = t0q3;
                const long long a = (d > 0) ? (term64(v, (d <= N) ? s0 : s1) + term64(prod[jl], s2)) : 0;
                acc[jl] = a;
                m |= abs64(a);
            }
            const int r = q_shift(chunk_bitlen(m, slot++));
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) toff[jl] = q16(acc[jl], r);
            eT = eref + r;
        }
        // Toffq row: 32 int16 of this thread straight to global memory
        if (p.Toff != nullptr && row_valid) {
            uint4* dst = reinterpret_cast<uint4*>(p.Toff + (chunk_id * kC + il) * kC + col0);
#pragma unroll
            for (int c = 0; c < 4; ++c)
                dst[c] = make_uint4(pack2(toff[8 * c + 0], toff[8 * c + 1]), pack2(toff[8 * c + 2], toff[8 * c + 3]),
                                    pack2(toff[8 * c + 4], toff[8 * c + 5]), pack2(toff[8 * c + 6], toff[8 * c + 7]));
        }
        if (row_valid && il == 0 && h == 0) p.t_exp[chunk_id] = eT;

        // ---- I9: Tbq = Q16(Toffq_ij beta_q_j); byte planes of the block-diagonal A operand of W / U
        int eTb;
        {
            long long acc[kHC];
            unsigned long long m = 0;
#pragma unroll
            for (int jl = 0; jl < kHC; ++jl) {
                acc[jl] = (long long)toff[jl] * sbeta[cb + col0 + jl];
                m |= abs64(acc[jl]);
            }
            const int r = q_shift(chunk_bitlen(m, slot++));
            uint32_t lo8[8], hi8[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t w0 = pack2(q16(acc[4 * i + 0], r), q16(acc[4 * i + 1], r));
                const uint32_t w1 = pack2(q16(acc[4 * i + 2], r), q16(acc[4 * i + 3], r));
                lo8[i] = plane_lo(w0, w1);
                hi8[i] = plane_hi(w0, w1);
            }
            eTb = eT - 15 + r;
            // row t's block occupies packed columns [cb/4, cb/4 + 16) of a 32-column plane; the other 16 are zero
            tmem_st8(lane_base + kAh + cb / 4 + h * 8, hi8);
            tmem_st8(lane_base + kAl + cb / 4 + h * 8, lo8);
#pragma unroll
            for (int i = 0; i < 8; ++i) lo8[i] = 0u;
            tmem_st8(lane_base + kAh + (16 - cb / 4) + h * 8, lo8);
            tmem_st8(lane_base + kAl + (16 - cb / 4) + h * 8, lo8);
            tmem_wait_st();
        }
        tc_fence_before_sync();
        cta_barrier();
        if (tid == 0) {
            // W accumulators = blockdiag(Tbq) Kq: M = 128, N = 128, K = 128 bytes per plane (4 steps of 32)
            tc_fence_after_sync();
            issue_ts(4, sPh_a, sPl_a, 4096, 16384, 1024, SWZ_128B);
        }

        // ---- I10: W, then U
        bool bad2 = false;
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
            const int xexp = (half == 0) ? kexp : vexp;
            // diagonal term beta_q_i * Xq_i for this thread's 64 columns, from its own row of the int16 tile (16 columns
            // at a time: the loops over the column blocks are not unrolled)
            const uint8_t* xtile = (half == 0) ? sK16 : sV16;
            auto load_x16 = [&](int c0, uint32_t (&w)[8]) {
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const uint4 v = *reinterpret_cast<const uint4*>(xtile + h * 16384 + t * 128 + ((((c0 >> 3) + c) ^ (t & 7)) << 4));
                    w[4 * c + 0] = v.x; w[4 * c + 1] = v.y; w[4 * c + 2] = v.z; w[4 * c + 3] = v.w;
                }
            };
            if (!wait_mma()) { bad2 = true; break; }
            tc_fence_after_sync();
            const int ep = eTb + xexp, ed = xexp - 15;
            const int eref = align_ref2(ep, ed);
            const int sp = ep - eref, sd = ed - eref;
            // The usual case: both terms are shifted left (their exponents are within the 16-bit window of each other), by
            // little enough that the shifts fold into 32-bit multipliers of the three accumulator words and of the key /
            // value mantissa: four widening multiply-adds per element instead of the recombination and two general shifts.
            const bool fold = sp >= 0 && sp <= 14 && sd >= 0 && sd <= 15;
            const int m_hh = fold ? (1 << (16 + sp)) : 0, m_mid = fold ? (1 << (8 + sp)) : 0, m_ll = fold ? (1 << sp) : 0;
            const int bqs = fold ? (bq << sd) : 0;
            // pass 1: the scale (bit length of the largest magnitude over the chunk's C x d block)
            unsigned long long m = 0;
#pragma unroll 1
            for (int c0 = 0; c0 < 64; c0 += 16) {
                uint32_t xr[8];
                load_x16(c0, xr);
                uint32_t dhh[16], dmid[16], dll[16];
                tmem_ld16(lane_base + kDhh + h * 64 + c0, dhh);
                tmem_ld16(lane_base + kDmid + h * 64 + c0, dmid);
                tmem_ld16(lane_base + kDll + h * 64 + c0, dll);
                tmem_wait_ld();
                if (DBG && dbg_row != nullptr) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) dbg_row[8 * kC + half * kD + h * 64 + c0 + i] = combine(dhh[i], dmid[i], dll[i]);
                }
                if (fold) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const uint32_t xw = xr[i >> 1];
                        const int x = (i & 1) ? hi16(xw) : lo16(xw);
                        const long long v = (long long)static_cast<int>(dhh[i]) * m_hh + (long long)static_cast<int>(dmid[i]) * m_mid +
                                            (long long)static_cast<int>(dll[i]) * m_ll + (long long)x * bqs;
                        m |= abs64(v);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const long long pr = combine(dhh[i], dmid[i], dll[i]);
                        const uint32_t xw = xr[i >> 1];
                        const int x = (i & 1) ? hi16(xw) : lo16(xw);
                        m |= abs64(term64(pr, sp) + term64((long long)bq * x, sd));
                    }
                }
            }
            const int rr = q_shift(chunk_bitlen(m, slot++));
            if (row_valid && il == 0 && h == 0) ((half == 0) ? p.w_exp : p.u_exp)[chunk_id] = eref + rr;
            // pass 2: mantissas, 64 int16 of this thread's row straight to global memory
            int16_t* out = ((half == 0) ? p.W : p.U) + grow * kD + h * 64;
#pragma unroll 1
            for (int c0 = 0; c0 < 64; c0 += 16) {
                uint32_t xr[8];
                load_x16(c0, xr);
                uint32_t dhh[16], dmid[16], dll[16];
                tmem_ld16(lane_base + kDhh + h * 64 + c0, dhh);
                tmem_ld16(lane_base + kDmid + h * 64 + c0, dmid);
                tmem_ld16(lane_base + kDll + h * 64 + c0, dll);
                tmem_wait_ld();
                uint32_t o[8];
                if (fold) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t xw = xr[i];
                        const long long v0 = (long long)static_cast<int>(dhh[2 * i]) * m_hh + (long long)static_cast<int>(dmid[2 * i]) * m_mid +
                                             (long long)static_cast<int>(dll[2 * i]) * m_ll + (long long)lo16(xw) * bqs;
                        const long long v1 = (long long)static_cast<int>(dhh[2 * i + 1]) * m_hh + (long long)static_cast<int>(dmid[2 * i + 1]) * m_mid +
                                             (long long)static_cast<int>(dll[2 * i + 1]) * m_ll + (long long)hi16(xw) * bqs;
                        o[i] = pack2(q16(v0, rr), q16(v1, rr));
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t xw = xr[i];
                        const long long v0 = term64(combine(dhh[2 * i], dmid[2 * i], dll[2 * i]), sp) + term64((long long)bq * lo16(xw), sd);
                        const long long v1 = term64(combine(dhh[2 * i + 1], dmid[2 * i + 1], dll[2 * i + 1]), sp) + term64((long long)bq * hi16(xw), sd);
                        o[i] = pack2(q16(v0, rr), q16(v1, rr));
                    }
                }
                if (row_valid) {
                    uint4* dst = reinterpret_cast<uint4*>(out + c0);
#pragma unroll
                    for (int c = 0; c < 2; ++c) dst[c] = make_uint4(o[4 * c], o[4 * c + 1], o[4 * c + 2], o[4 * c + 3]);
                }
            }
            if (half == 0) {
                tc_fence_before_sync();
                cta_barrier();  // the W accumulators, the K planes and the int16 K tile have been read by everyone
                if (tid == 0) {
                    if (has_next) {
                        const TileCoord nc = decode_tile(next, p);
                        mbar_arrive_expect_tx(&bar_k, 32768);
                        tma_load_3d(sK16, &tmK, &bar_k, 0, nc.t0, nc.bhk);
                        tma_load_3d(sK16 + 16384, &tmK, &bar_k, 64, nc.t0, nc.bhk);
                    }
                    if (!wait_bar(&bar_v, par_kv)) set_fail();
                }
                cta_barrier();  // the V tile has arrived (or the wait failed)
                if (failed()) { bad2 = true; break; }
                split_planes(sV16);
                fence_proxy_async_smem();
                tc_fence_before_sync();
                cta_barrier();
                if (tid == 0) {
                    tc_fence_after_sync();
                    issue_ts(4, sPh_a, sPl_a, 4096, 16384, 1024, SWZ_128B);
                }
            }
        }
        if (bad2) break;
        par_kv ^= 1;
    }
    if (failed() && tid == 0) atomicExch(p.status, GDN_ERR_TIMEOUT);

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

// [heads][T][128] 16-bit tensor, boxes of 128 rows x 64 columns (128-byte lines), 128-byte swizzle
bool make_map16(CUtensorMap* tm, const void* base, long long heads, int T) {
    EncodeTiledFn enc = get_encode_fn();
    if (enc == nullptr) return false;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(kD), static_cast<cuuint64_t>(T), static_cast<cuuint64_t>(heads)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(kD) * 2, static_cast<cuuint64_t>(T) * kD * 2};
    cuuint32_t box[3] = {64, 128, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT16, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

int launch_tc_int16(const ProblemI16& q, cudaStream_t stream) {
    if (q.C != kC || q.d_k != kD || q.d_v != kD) return GDN_ERR_UNSUPPORTED;
    if (q.order < 1 || q.order > 3 || q.steps < 0 || q.steps > kSMax) return GDN_ERR_UNSUPPORTED;
    if ((long long)q.B * q.H_v * q.T == 0) return GDN_OK;
    int* status = device_status_word();
    if (status == nullptr) return GDN_ERR_LAUNCH;
    CUtensorMap mK, mV;
    const long long hk = (long long)q.B * q.H_k, hv = (long long)q.B * q.H_v;
    if (!make_map16(&mK, q.Kq, hk, q.T) || !make_map16(&mV, q.Vq, hv, q.T)) return GDN_ERR_LAUNCH;
    ParamsI16 prm;
    prm.beta_q = q.beta_q;
    prm.decay_q = q.decay_q;
    prm.k_exp = q.k_exp;
    prm.v_exp = q.v_exp;
    prm.W = q.Wq;
    prm.U = q.Uq;
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
    prm.n_tiles = (long long)q.B * q.H_v * prm.n_tt;
    if (prm.n_tiles >= (1LL << 31) - 4096) return GDN_ERR_UNSUPPORTED;
    int8_decay_lut(prm.lut);
    const int smem = kSmemTotal + 1024;
    auto kern = (prm.dbg != nullptr) ? chunk_tc_int16_kernel<true> : chunk_tc_int16_kernel<false>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return GDN_ERR_LAUNCH;
    const long long grid = prm.n_tiles < 148 ? prm.n_tiles : 148;
    kern<<<static_cast<int>(grid), kThreads, smem, stream>>>(mK, mV, prm);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_LAUNCH;
}

}  // namespace gdn
