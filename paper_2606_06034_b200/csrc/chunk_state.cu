// State passing and output of chunk-wise Gated DeltaNet, given W (gated) and U of every chunk (tcgen05 + TMEM + TMA).
//
// What it computes, per (batch, value head), chunk after chunk (C = 64 tokens, S0 = state [d_v x d_k] carried in,
// g = chunk-local cumulative log-gate, W = T diag(beta exp(g)) K, U = T diag(beta) V from the chunk-prepare path):
//     U_new = U - W S0^T
//     o_i   = scale (exp(g_i) S0 q_i + sum_{j <= i} exp(g_i - g_j) <k_j, q_i> U_new_j)
//     S_end = exp(g_C) S0 + sum_j exp(g_C - g_j) U_new_j k_j^T
// This is the WY form of the gated delta rule that the chunk-prepare quantities exist for (Sec. 2.1); the chunks of
// one head are a serial chain, heads are independent.
//
// Everything is evaluated with the value dimension on the 128 TMEM lanes ("transposed"): one CTA per (batch, head)
// keeps the state S [d_v x d_k] as an fp32 accumulator in TMEM for the whole sequence, lane t = value feature t.
//     D1  = S0 W^T - U^T      A = S0 as hi + lo bf16 halves in TMEM (the state is O(1) while U_new can be small:
//                             a single bf16 copy costs 1e-2 on strongly correlated keys), B = W tile; the
//                             transpose of U comes from the tensor core as
//                             (-I) U^T with a constant A operand, so no thread ever transposes anything
//     PT  = K Q^T             lanes 0..63 = token j, columns = token i
//     O1  = S0 Q^T
//     O2  = U_new^T P^T       A = bf16(U_new^T) (written over D1's columns), B = P_ij = exp(g_i-g_j) PT_ji [j <= i]
//     S  += (U_new^T exp(g_C - g_j)) K     accumulated onto exp(g_C) S0 (the decay is a pass over the TMEM columns)
//     O^T = scale (exp(g_i) O1 + O2)  -> transposed through shared memory -> bulk tensor store
// Two MMA groups per chunk; Q, K, W, U tiles of the next chunk are in flight (two stages) while a chunk is worked on.
// All operand layouts are the ones the chunk-prepare kernel uses.
// Warps: 16 compute warps (four threads per TMEM lane), one that issues every MMA, one that issues the TMA loads and
// the output stores. The chain of a sequence is thread work (every phase runs on all 16 warps at once, so its
// instruction count is what it costs); hand-offs to the issuing warp are hardware barriers, completions come back
// through mbarriers (a poll costs ~200 cycles, so as few as possible are waited for).
// Instantiations: packed variable-length sequences (one CTA per (sequence, value head), starting at the sequence's
// first token; the tokens a short last chunk lacks decay nothing and write nothing); state only (no queries, no
// output: the first pass of the segmented call for few long sequences, see launch_chunk_state_segmented); keys and
// queries L2-normalised here (GDN_FLAG_K_L2NORM).
#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace gdn {
namespace {

using namespace sm100;

constexpr int kC = 64;         // chunk size
constexpr int kD = 128;        // d_k = d_v
constexpr int kThreads = 512;  // compute threads, four per TMEM lane; two more warps issue the MMAs and the TMA loads
constexpr float kLog2e = 1.4426950408889634f;

// TMEM column map (512 columns: one CTA per SM)
constexpr uint32_t kSD = 0;    // 128: state S, fp32 accumulator
constexpr uint32_t kSA = 128;  // 64: bf16(S0) as A operand (K = d_k)
constexpr uint32_t kIA = 192;  // 64: -I as A operand (K = d_v), constant
constexpr uint32_t kD1 = 256;  // 64: S0 W^T - U^T, then the two bf16 forms of U_new^T as A operands
constexpr uint32_t kPT = 320;  // 64: K Q^T (lanes 0..63); once read, the lo bf16 halves of the two forms of U_new^T
constexpr uint32_t kO1 = 384;  // 64: S0 Q^T
constexpr uint32_t kO2 = 448;  // 64: U_new^T P^T; between chunks it holds the lo bf16 half of S0 (A operand)
constexpr uint32_t kTmemCols = 512;

// shared memory map (bytes; 1 KB aligned). A [64 x 128] bf16 tile is two [64 x 64] sub-tiles of 8 KB (128B swizzle).
constexpr int kTileBytes = 16384;
constexpr int kStageBytes = 4 * kTileBytes;  // Q, K, W, U
constexpr int kOffQ = 0, kOffK = kTileBytes, kOffW = 2 * kTileBytes, kOffU = 3 * kTileBytes;
constexpr int kOffP = 2 * kStageBytes;       // 2 x 8 KB: P as B operand [64 x 64] (MN-major, no swizzle), hi and lo halves
constexpr int kOffO = kOffP + 16384;          // 2 x 16 KB: O tile staged for the bulk store (128B swizzle), two buffers
constexpr int kTab = 5 * 64;  // floats per table buffer: exp(g_i), exp(g_C - g_j), g, 1 / ||k_j||, 1 / ||q_i||
constexpr int kOffG = kOffO + 2 * kTileBytes;  // three table buffers
constexpr int kSmemTotal = kOffG + 3 * kTab * 4;


struct ParamsS {
    const float* g;
    const float* S_in;  // may be null
    float* S_out;       // may be null
    int* status;
    int H_k, H_v, T, group;
    float scale;
    unsigned flags;  // GDN_FLAG_G_RAW: g holds raw log-gates, prefix-summed inside every chunk here
    // packed variable-length sequences (B = 1): sequence s holds the tokens [seq_start[s], seq_end[s]) of tensors
    // with T tokens per head and is chunked from its own first token; null for dense tensors
    const int* seq_start;  // first token of sequence s
    const int* seq_end;    // one past its last token (the public call passes cu_seqlens and cu_seqlens + 1)
    const int* seq_no_u;   // optional: sequence s runs with U = 0 (the state map of a segment, see the segmented call)
    __nv_bfloat16* O;  // output tensor (rows of a short last chunk are stored one by one)
};

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// bounded mbarrier wait (about a second), as in the chunk-prepare kernels
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t i = 0;
    while (!mbar_try_wait_hint(bar, parity, 2000u)) {
        if ((++i & 63u) == 0 && clock64() - t0 > 2000000000LL) return false;
    }
    return true;
}

// Hand-off from the 512 compute threads to the issuing warp over a hardware barrier: the threads arrive and go on, the
// issuing warp waits. (An mbarrier poll costs the waiting warp ~200-300 cycles per hand-off on the chain of the
// sequence; this is a few tens.) The wait has no bound of its own: threads whose own bounded waits run out arrive on both hand-offs before they leave.
template <int ID>
__device__ __forceinline__ void handoff_arrive() {
    asm volatile("bar.arrive %0, %1;" ::"n"(ID), "n"(kThreads + 32) : "memory");
}
template <int ID>
__device__ __forceinline__ void handoff_wait() {
    asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(kThreads + 32) : "memory");
}

// VAR: packed variable-length sequences (own instantiation: its masks sit on the chain the dense case is bound by)
// SO: state only: no queries, no output (the first pass of the segmented call); U may be absent per sequence.
// NRM: GDN_FLAG_K_L2NORM (keys and queries normalised here): own instantiations, the plain chain pays nothing for it.
template <bool VAR, bool SO, bool NRM>
__global__ void __launch_bounds__(kThreads + 64, 1)
chunk_state_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmU,
                   const __grid_constant__ CUtensorMap tmO, const ParamsS p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    float* gtab = reinterpret_cast<float*>(smem + kOffG);  // per buffer: exp(g_i), exp(g_C - g_j), g_i, 1/||k||, 1/||q|| (64 each)

    // One mbarrier per MMA group that is waited for (never two pending phases on one barrier), two per-stage TMA
    // barriers, and two on which the storing warp releases the output staging buffers. The hand-offs from the 512
    // compute threads to the issuing and the storing warp go over hardware barriers 4, 5 and 6 (handoff_arrive / _wait).
    __shared__ uint64_t bar_full[2], bar_pre, bar_d1, bar_o2, bar_g2, bar_stg[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int s_fail;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int t = tid & 127;  // TMEM lane: value feature (state rows, output columns); token j for PT
    const int h = (tid >> 7) & 3;  // column quarter: 16 of the 64 columns of a product, 32 of the 128 state columns
    const int wq = warp & 3;
    const int lane = tid & 31;
    const bool issuer = warp == kThreads / 32;        // every tcgen05.mma
    const bool producer = warp == kThreads / 32 + 1;  // every TMA load

    if (tid == 0) {
        mbar_init(&bar_full[0], 1);
        mbar_init(&bar_full[1], 1);
        mbar_init(&bar_pre, 1);
        mbar_init(&bar_d1, 1);
        mbar_init(&bar_o2, 1);
        mbar_init(&bar_g2, 1);
        mbar_init(&bar_stg[0], 1);
        mbar_init(&bar_stg[1], 1);
        s_fail = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmW);
        tma_prefetch_desc(&tmU);
        tma_prefetch_desc(&tmO);
    }
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_s;
    const uint32_t lane_base = tmem + (static_cast<uint32_t>(wq * 32) << 16);

    // dense: one CTA per (batch, value head), bhv = row of the [B * H_v, T] tensors. Packed sequences: one CTA per
    // (sequence, value head); the tensors have one batch row per head and the sequence starts at token tok0
    const int b = blockIdx.x / p.H_v, hv = blockIdx.x - b * p.H_v;
    const int tok0 = VAR ? __ldg(p.seq_start + b) : 0;
    const int len = VAR ? __ldg(p.seq_end + b) - tok0 : p.T;
    const bool no_u = SO && p.seq_no_u != nullptr && __ldg(p.seq_no_u + b) != 0;
    const int bhv = VAR ? hv : blockIdx.x;
    const int bhk = VAR ? hv / p.group : b * p.H_k + hv / p.group;
    // Token-major tensors [B, T, H, d] (GDN_FLAG_LAYOUT_BTHD) are seen by TMA as (H * d, T, B): the head picks the first
    // column of a box, the batch its outermost index; consecutive tokens of g are H_v apart.
    const bool bthd = (p.flags & GDN_FLAG_LAYOUT_BTHD) != 0;
    const int bz = VAR ? 0 : b;
    const int kx = bthd ? (hv / p.group) * kD : 0, kz = bthd ? bz : bhk;  // Q, K boxes
    const int vx = bthd ? hv * kD : 0, vz = bthd ? bz : bhv;              // W, U, O boxes
    const long long grow0 = bthd ? ((long long)bz * p.T + tok0) * p.H_v + hv : (long long)bhv * p.T + tok0;  // first token's row
    const int gstep = bthd ? p.H_v : 1;
    const int n_c = (len + kC - 1) / kC;
    const float* gseq = p.g + grow0;
    const uint32_t smem_a = smem_u32(smem);
    volatile int* fail = reinterpret_cast<volatile int*>(&s_fail);

    if (producer) {
        // ================= loading / storing warp: the four tiles of chunk c into stage c & 1, as soon as the products
        // that read the stage's previous tiles are complete; and the bulk stores of the staged output tiles, so that
        // no compute thread waits for the others at the end of a chunk
        const bool lead = elect_one();
        auto load_stage = [&](int c) {
            uint8_t* st = smem + (c & 1) * kStageBytes;
            uint64_t* bar = &bar_full[c & 1];
            mbar_arrive_expect_tx(bar, SO ? 3 * kTileBytes : kStageBytes);
            const int t0 = tok0 + c * kC;
            if (!SO) {
                tma_load_3d(st + kOffQ, &tmQ, bar, kx, t0, kz);
                tma_load_3d(st + kOffQ + 8192, &tmQ, bar, kx + 64, t0, kz);
            }
            tma_load_3d(st + kOffK, &tmK, bar, kx, t0, kz);
            tma_load_3d(st + kOffK + 8192, &tmK, bar, kx + 64, t0, kz);
            tma_load_3d(st + kOffW, &tmW, bar, vx, t0, vz);
            tma_load_3d(st + kOffW + 8192, &tmW, bar, vx + 64, t0, vz);
            tma_load_3d(st + kOffU, &tmU, bar, vx, t0, vz);
            tma_load_3d(st + kOffU + 8192, &tmU, bar, vx + 64, t0, vz);
        };
        if (lead) {
            if (n_c > 0) load_stage(0);
            if (n_c > 1) load_stage(1);
        }
        uint32_t par = 0;
        for (int c = 0; c < n_c && *fail == 0; ++c) {
            // the staged output tile of chunk c is complete (every compute thread has arrived)
            if (!SO) handoff_wait<6>();
            if (lead && *fail == 0) {
                if (!SO && !(VAR && len - c * kC < kC)) {  // (a short last chunk is stored row by row by the compute threads)
                    tma_store_3d(&tmO, smem + kOffO + (c & 1) * kTileBytes, vx, tok0 + c * kC, vz);
                    tma_store_3d(&tmO, smem + kOffO + (c & 1) * kTileBytes + 8192, vx + 64, tok0 + c * kC, vz);
                    tma_store_commit();
                }
                if (c + 2 < n_c) {
                    if (!wait_bar(&bar_g2, par)) *fail = 1;
                    if (*fail == 0) load_stage(c + 2);
                }
                if (!SO) {
                    tma_store_wait_read<0>();
                    mbar_arrive(&bar_stg[c & 1]);  // the staging buffer may be written again (chunk c + 2)
                }
            }
            par ^= 1;
            __syncwarp();
        }
        if (lead) tma_store_wait_all<0>();
        __syncwarp();
    } else if (issuer) {
        // ================= issuing warp: every tcgen05.mma, in the order the tensor pipe runs them
        const uint32_t idesc_kk64 = instr_desc(128, 64, 1, 1, 0, 0, 1);   // B K-major (a TMA tile as [N x K])
        const uint32_t idesc_mn64 = instr_desc(128, 64, 1, 1, 0, 1, 1);   // B MN-major
        const uint32_t idesc_mn128 = instr_desc(128, 128, 1, 1, 0, 1, 1);
        // the products of chunk c that do not depend on the state: D1 <- (-I) U^T and PT = K Q^T
        auto issue_pre = [&](int c) {
            const uint32_t sa = smem_a + (c & 1) * kStageBytes;
            if (!wait_bar(&bar_full[c & 1], (c >> 1) & 1)) *fail = 1;
            tc_fence_after_sync();
            if (*fail == 0 && elect_one()) {
                if (!no_u) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint64_t bd = smem_desc(sa + kOffU + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024, SWZ_128B);
                        mma_f16_ts(tmem + kD1, tmem + kIA + ks * 8, bd, idesc_kk64, ks > 0);
                    }
                }
                if (!SO) {
                    // rows 64..127 of the A operand read past the 64-row K tile: unused lanes
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint64_t ad = smem_desc(sa + kOffK + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024, SWZ_128B);
                        const uint64_t bd = smem_desc(sa + kOffQ + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024, SWZ_128B);
                        mma_f16_ss(tmem + kPT, ad, bd, idesc_kk64, ks > 0);
                    }
                    mma_commit(&bar_pre);  // (state only: nothing of this group is waited for by itself)
                }
            }
            __syncwarp();
        };
        for (int c = 0; c < n_c && *fail == 0; ++c) {
            const uint32_t st_a = smem_a + (c & 1) * kStageBytes;
            // the state copies (and, for the first chunk, the constant operand) are in place
            handoff_wait<4>();
            tc_fence_after_sync();
            if (c == 0) issue_pre(0);
            if (*fail == 0 && elect_one()) {
                // D1 += (S0_hi + S0_lo) W^T onto -U^T, with its own completion barrier
#pragma unroll
                for (int part = 0; part < 2; ++part) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint64_t bd = smem_desc(st_a + kOffW + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024, SWZ_128B);
                        mma_f16_ts(tmem + kD1, tmem + (part == 0 ? kSA : kO2) + ks * 8, bd, idesc_kk64,
                                   !no_u || part > 0 || ks > 0);
                    }
                }
                mma_commit(&bar_d1);
                if (!SO) {
                    // O1 = (S0_hi + S0_lo) Q^T
#pragma unroll
                    for (int part = 0; part < 2; ++part) {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            const uint64_t bd = smem_desc(st_a + kOffQ + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024, SWZ_128B);
                            mma_f16_ts(tmem + kO1, tmem + (part == 0 ? kSA : kO2) + ks * 8, bd, idesc_kk64, part > 0 || ks > 0);
                        }
                    }
                }
                // (no completion barrier of its own: the commit behind the output product below covers it, and a wait
                // costs the threads ~200 cycles even on a completed phase)
            }
            __syncwarp();
            // U_new^T (hi, lo; plain, scaled), P (hi, lo) and the decayed accumulator are in place
            handoff_wait<5>();
            tc_fence_after_sync();
            if (*fail == 0 && elect_one()) {
                if (!SO) {
                    // O2 = U_new^T P^T = Uh Ph + Ul Ph + Uh Pl (K-dim = 64 tokens; the plain copy of tokens 16 ks.. sits
                    // at columns 16 ks .. 16 ks + 7 of its region, the gate-scaled one at 16 ks + 8 ..)
#pragma unroll
                    for (int part = 0; part < 3; ++part) {
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const uint64_t bd = smem_desc(smem_a + kOffP + (part == 2 ? 8192 : 0) + ks * 256, 128, 1024, SWZ_NONE);
                            mma_f16_ts(tmem + kO2, tmem + (part == 1 ? kPT : kD1) + ks * 16, bd,
                                       idesc_mn64, part > 0 || ks > 0);
                        }
                    }
                    mma_commit(&bar_o2);  // the output is finished while the state update still runs
                }
                // S += (U_new^T exp(g_C - g_j)) K, hi + lo (the K tile as MN-major operand, N = 128)
#pragma unroll
                for (int part = 0; part < 2; ++part) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        const uint64_t bd = smem_desc(st_a + kOffK + ks * 2048, 8192, 1024, SWZ_128B);
                        mma_f16_ts(tmem + kSD, tmem + (part == 0 ? kD1 : kPT) + ks * 16 + 8, bd,
                                   idesc_mn128, true);
                    }
                }
                mma_commit(&bar_g2);
            }
            __syncwarp();
            // D1 and PT are only read by the products just issued, which the tensor pipe runs first: the
            // state-independent products of the next chunk follow them directly
            if (c + 1 < n_c) issue_pre(c + 1);
        }
    } else {
        // ================= compute threads (512): four per TMEM lane
        uint32_t par_pre = 0, par_d1 = 0, par_o2 = 0, par_g2 = 0;
        // completion of an MMA group: every lane polls the mbarrier (no CTA-wide barrier on this path). A poll of a
        // completed phase costs ~200 cycles whoever issues it; polling from lane 0 alone added a divergent branch and a
        // shuffle, ~150 cycles more per wait.
        auto wait_group = [&](uint64_t* bar, uint32_t& par) -> bool {
            const bool good = wait_bar(bar, par);
            if (!good) *fail = 1;
            par ^= 1;
            tc_fence_after_sync();
            return good;
        };
        // ---- constant A operand -I, initial state, and its bf16 copies (hi in kSA, lo in kO2)
        {
            uint32_t r[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int col = h * 16 + i;  // packed column: features 2 col, 2 col + 1
                r[i] = (col == (t >> 1)) ? ((t & 1) ? 0xBF800000u : 0x0000BF80u) : 0u;
            }
            tmem_st16(lane_base + kIA + h * 16, r);
            // this thread's quarter of state row t: columns [32 h, 32 h + 32)
            const float* s0 = (p.S_in != nullptr) ? p.S_in + ((long long)blockIdx.x * kD + t) * kD + h * 32 : nullptr;
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                uint32_t v[16], pk[8];
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = (s0 != nullptr) ? __float_as_uint(__ldg(s0 + part * 16 + i)) : 0u;
                tmem_st16(lane_base + kSD + h * 32 + part * 16, v);
#pragma unroll
                for (int i = 0; i < 8; ++i) pk[i] = pack_bf16x2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
                tmem_st8(lane_base + kSA + h * 16 + part * 8, pk);
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    pk[i] = pack_bf16x2(__uint_as_float(v[2 * i]) - bf16_lo(pk[i]), __uint_as_float(v[2 * i + 1]) - bf16_hi(pk[i]));
                tmem_st8(lane_base + kO2 + h * 16 + part * 8, pk);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            handoff_arrive<4>();
        }
        // gates of the first chunk
        float g_reg = 0.f;
        // (a short last chunk: tokens past the sequence's end decay nothing and write nothing)
        // The gate tables are the job of threads 64..127: their lanes hold no row of P, so they are idle while the other
        // half of the CTA forms P.
        const int tt = tid - 64;  // token of a table thread
        const bool tabler = tt >= 0 && tt < 64;
        if (n_c > 0 && tabler) g_reg = (!VAR || tt < len) ? __ldg(gseq + tt * gstep) : 0.f;
        bool ok = true;
        // gate tables of a chunk: written by 64 threads into the buffer of that chunk one barrier before they are read
        const bool g_raw = (p.flags & GDN_FLAG_G_RAW) != 0;
        constexpr bool f_nrm = NRM;
        auto fill_tables = [&](int c) {
            if (tabler) {
                float* tb = gtab + (c % 3) * kTab;
                float gc = g_reg;
                const int left = len - c * kC;  // tokens of this chunk (>= 64 except for a short last chunk)
                if (g_raw) {
                    // inclusive prefix sum over the chunk's 64 tokens: inside each of the two warps by shuffles ...
#pragma unroll
                    for (int off = 1; off < 32; off <<= 1) {
                        const float v = __shfl_up_sync(0xFFFFFFFFu, gc, off);
                        if (lane >= off) gc += v;
                    }
                    if (tt == 31) tb[128 + 63] = gc;  // ... and the first warp's total through the table itself
                    asm volatile("bar.sync 3, 64;" ::: "memory");
                    if (tt >= 32) gc += tb[128 + 63];
                    asm volatile("bar.sync 3, 64;" ::: "memory");
                }
                tb[128 + tt] = gc;
                asm volatile("bar.sync 3, 64;" ::: "memory");
                if (VAR && !g_raw && left < kC) {
                    // cumulative gates: tokens past the end keep the gate of the last real token
                    gc = tb[128 + (tt < left ? tt : left - 1)];
                    asm volatile("bar.sync 3, 64;" ::: "memory");
                    tb[128 + tt] = gc;
                    asm volatile("bar.sync 3, 64;" ::: "memory");
                }
                const float gC = tb[128 + 63];  // cumulative gate of the chunk's last token
                // (with the keys and queries normalised here, their factors ride on the two gate factors: exp(g_i) only
                // ever multiplies a product with q_i, exp(g_C - g_j) one with k_j)
                tb[tt] = fast_exp2(gc * kLog2e) * (f_nrm ? tb[256 + tt] : 1.f);
                tb[64 + tt] = fast_exp2((gC - gc) * kLog2e) * (f_nrm ? tb[192 + tt] : 1.f);
            }
        };
        // GDN_FLAG_K_L2NORM: 1 / ||k_j|| and 1 / ||q_i|| of chunk c from its tiles in shared memory, by the 256 threads
        // whose lanes hold no row of P (the sum of squares of a row does not care about the swizzle inside the row)
        auto fill_norms = [&](int c) {
            if (wq >= 2) {
                // (the issuing warp has waited for these tiles, or will; observing the phase here orders the reads below)
                if (!wait_bar(&bar_full[c & 1], (c >> 1) & 1)) *fail = 1;
                const int u = (tid >> 7) * 64 + (tid & 63);  // 0 .. 255
                float* tb = gtab + (c % 3) * kTab;
                // A warp reads 512 contiguous bytes per step (four rows of a 64-column sub-tile): conflict-free. Thread u
                // sees rows u >> 3 and 32 + (u >> 3) of both sub-tiles; the eight lanes of a row add up by shuffles.
#pragma unroll
                for (int which = 0; which < (SO ? 1 : 2); ++which) {
                    const uint8_t* tile = smem + (c & 1) * kStageBytes + (which == 0 ? kOffK : kOffQ) + u * 16;
                    float acc[2] = {0.f, 0.f};
#pragma unroll
                    for (int it = 0; it < 4; ++it) {
                        const uint4 w4 = *reinterpret_cast<const uint4*>(tile + (it >> 1) * 8192 + (it & 1) * 4096);
                        const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float a = __uint_as_float(w[i] << 16), b = __uint_as_float(w[i] & 0xFFFF0000u);
                            acc[it & 1] = fmaf(a, a, fmaf(b, b, acc[it & 1]));
                        }
                    }
#pragma unroll
                    for (int off = 1; off < 8; off <<= 1) {
                        acc[0] += __shfl_xor_sync(0xFFFFFFFFu, acc[0], off);
                        acc[1] += __shfl_xor_sync(0xFFFFFFFFu, acc[1], off);
                    }
                    if ((u & 7) == 0) {
                        tb[(which == 0 ? 192 : 256) + (u >> 3)] = rsqrtf(fmaxf(acc[0], 1e-30f));
                        tb[(which == 0 ? 192 : 256) + 32 + (u >> 3)] = rsqrtf(fmaxf(acc[1], 1e-30f));
                    }
                }
                asm volatile("bar.sync 7, 256;" ::: "memory");
            }
        };
        if (n_c > 0) {
            if (f_nrm) fill_norms(0);
            fill_tables(0);
        }
        asm volatile("bar.sync 1, 512;" ::: "memory");
        for (int c = 0; c < n_c; ++c) {
            const float* se = gtab + (c % 3) * kTab;  // exp(g_i)
            const float* sf = se + 64;               // exp(g_C - g_j)
            const float* sg = se + 128;              // g_i (cumulative inside the chunk)
            const float gC = sg[63];
            const int left = len - c * kC;
            const bool short_chunk = VAR && left < kC;
            if (c + 1 < n_c && tabler) g_reg = (!VAR || (c + 1) * kC + tt < len) ? __ldg(gseq + ((c + 1) * kC + tt) * gstep) : 0.f;

            // ---- decay of the accumulator, S <- exp(g_C) S0 (the products of this chunk read the bf16 copies)
            {
                const float dec = fast_exp2(gC * kLog2e);
                uint32_t v[32];
                tmem_ld32(lane_base + kSD + h * 32, v);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * dec);
                uint32_t w16[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) w16[i] = v[i];
                tmem_st16(lane_base + kSD + h * 32, w16);
#pragma unroll
                for (int i = 0; i < 16; ++i) w16[i] = v[16 + i];
                tmem_st16(lane_base + kSD + h * 32 + 16, w16);
            }
            // ---- P_ij = exp(g_i - g_j) PT_ji for j <= i (hi + lo): token j = lane (rows 0..63 only), this thread's 16 columns i
            if (!SO && !wait_group(&bar_pre, par_pre)) { ok = false; break; }
            if (!SO && wq < 2) {
                uint32_t d[16];
                tmem_ld16(lane_base + kPT + h * 16, d);
                tmem_wait_ld();
                const float gj = sg[t] * kLog2e;
                const float rkj = f_nrm ? sg[64 + t] : 1.f;
                float gi16[16];  // g of this thread's 16 columns (four 16-byte loads instead of sixteen scalar ones)
#pragma unroll
                for (int i4 = 0; i4 < 4; ++i4) {
                    const float4 q4 = *reinterpret_cast<const float4*>(sg + h * 16 + i4 * 4);
                    gi16[i4 * 4 + 0] = q4.x; gi16[i4 * 4 + 1] = q4.y; gi16[i4 * 4 + 2] = q4.z; gi16[i4 * 4 + 3] = q4.w;
                }
#pragma unroll
                for (int c2 = 0; c2 < 2; ++c2) {
                    uint32_t w[4], wl[4];
#pragma unroll
                    for (int i2 = 0; i2 < 4; ++i2) {
                        float v[2];
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const int i = h * 16 + c2 * 8 + i2 * 2 + q;
                            float x = __uint_as_float(d[c2 * 8 + i2 * 2 + q]) *
                                      fast_exp2(fminf(fmaf(gi16[c2 * 8 + i2 * 2 + q], kLog2e, -gj), 0.f));
                            if (f_nrm) x *= rkj * sg[128 + i];  // 1 / (||k_j|| ||q_i||)
                            v[q] = (t <= i) ? x : 0.f;
                        }
                        w[i2] = pack_bf16x2(v[0], v[1]);
                        wl[i2] = pack_bf16x2(v[0] - bf16_lo(w[i2]), v[1] - bf16_hi(w[i2]));
                    }
                    // B operand [K-dim = j][N = i], MN-major, no swizzle: the 16-byte piece of row j for column group n8
                    *reinterpret_cast<uint4*>(smem + kOffP + (h * 2 + c2) * 1024 + t * 16) = make_uint4(w[0], w[1], w[2], w[3]);
                    *reinterpret_cast<uint4*>(smem + kOffP + 8192 + (h * 2 + c2) * 1024 + t * 16) = make_uint4(wl[0], wl[1], wl[2], wl[3]);
                }
            }
            // the next chunk's gate tables, by threads that had no part in P (published by the barrier at the chunk's end)
            if (c + 1 < n_c && !f_nrm) fill_tables(c + 1);
            // ---- U_new^T = -D1 as bf16 hi + lo, plain and gate-scaled (the sums over the tokens of a chunk telescope
            // on correlated keys, so single bf16 copies cost 1e-2 there). This thread's 16 tokens are one k-step of the
            // products that consume them: the hi halves are written over its own D1 columns (plain -> 16 h .. 16 h + 7,
            // scaled -> 16 h + 8 ..), the lo halves at the same offsets of the PT region (read above by this thread).
            if (!wait_group(&bar_d1, par_d1)) { ok = false; break; }
            {
                uint32_t d[16];
                tmem_ld16(lane_base + kD1 + h * 16, d);
                tmem_wait_ld();
                uint32_t hi[16], lo[16];
#pragma unroll
                float f16[16];
#pragma unroll
                for (int i4 = 0; i4 < 4; ++i4) {
                    const float4 q4 = *reinterpret_cast<const float4*>(sf + h * 16 + i4 * 4);
                    f16[i4 * 4 + 0] = q4.x; f16[i4 * 4 + 1] = q4.y; f16[i4 * 4 + 2] = q4.z; f16[i4 * 4 + 3] = q4.w;
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    float u0 = -__uint_as_float(d[2 * i]), u1 = -__uint_as_float(d[2 * i + 1]);
                    if (short_chunk) {  // rows past the sequence's end hold another sequence's W, U
                        if (h * 16 + 2 * i >= left) u0 = 0.f;
                        if (h * 16 + 2 * i + 1 >= left) u1 = 0.f;
                    }
                    const float s0 = u0 * f16[2 * i], s1 = u1 * f16[2 * i + 1];
                    hi[i] = pack_bf16x2(u0, u1);
                    hi[8 + i] = pack_bf16x2(s0, s1);
                    lo[i] = pack_bf16x2(u0 - bf16_lo(hi[i]), u1 - bf16_hi(hi[i]));
                    lo[8 + i] = pack_bf16x2(s0 - bf16_lo(hi[8 + i]), s1 - bf16_hi(hi[8 + i]));
                }
                tmem_st16(lane_base + kD1 + h * 16, hi);
                tmem_st16(lane_base + kPT + h * 16, lo);
            }
            fence_proxy_async_smem();
            tmem_wait_st();
            tc_fence_before_sync();
            handoff_arrive<5>();
            // with the norms of the next chunk's keys and queries in the tables, both are formed here instead: the next
            // chunk's tiles are still on their way while P is formed, and the threads idle now anyway
            if (c + 1 < n_c && f_nrm) {
                fill_norms(c + 1);
                fill_tables(c + 1);
            }

            if (!SO) {
                // The storing warp has released the PREVIOUS chunk's staging buffer (polled here, in the shadow of the
                // output product; the store was issued most of a chunk ago). That is one chunk later than this chunk's
                // own buffer needs (chunk c - 2 used it, and the stores are read in order), but it also says that the
                // storing warp has taken the previous chunk's hand-off: the threads must not arrive on that hardware
                // barrier a second time before it has, however long a store may be held up.
                if (c >= 1 && !wait_bar(&bar_stg[(c - 1) & 1], ((c - 1) >> 1) & 1)) { *fail = 1; ok = false; break; }
                // ---- exp(g_i) O1 (complete with O2: products finish in the order they were issued)
                if (!wait_group(&bar_o2, par_o2)) { ok = false; break; }
                float o[16];
                {
                    uint32_t d[16];
                    tmem_ld16(lane_base + kO1 + h * 16, d);
                    tmem_wait_ld();
    #pragma unroll
                    for (int i4 = 0; i4 < 4; ++i4) {
                        const float4 e4 = *reinterpret_cast<const float4*>(se + h * 16 + i4 * 4);
                        o[i4 * 4 + 0] = __uint_as_float(d[i4 * 4 + 0]) * e4.x;
                        o[i4 * 4 + 1] = __uint_as_float(d[i4 * 4 + 1]) * e4.y;
                        o[i4 * 4 + 2] = __uint_as_float(d[i4 * 4 + 2]) * e4.z;
                        o[i4 * 4 + 3] = __uint_as_float(d[i4 * 4 + 3]) * e4.w;
                    }
                }
                // ---- O^T = scale (exp(g_i) O1 + O2): element (token i, feature t) of the staged tile
                {
                    uint32_t d[16];
                    tmem_ld16(lane_base + kO2 + h * 16, d);
                    tmem_wait_ld();
                    uint8_t* sub = smem + kOffO + (c & 1) * kTileBytes + (t >> 6) * 8192;
                    const int cch = (t & 63) >> 3;
    #pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int tok = h * 16 + i;
                        const __nv_bfloat16 v = __float2bfloat16_rn(p.scale * (o[i] + __uint_as_float(d[i])));
                        *reinterpret_cast<__nv_bfloat16*>(sub + tok * 128 + ((cch ^ (tok & 7)) << 4) + (t & 7) * 2) = v;
                    }
                }
                // the tile goes to the storing warp: no compute thread waits for the others here
                fence_proxy_async_smem();
                handoff_arrive<6>();
            }
            // ---- bf16 copies (hi, lo) of the new state for the next chunk's products; the lo half goes where O2 was
            // (this thread has read its O2 columns above)
            if (!wait_group(&bar_g2, par_g2)) { ok = false; break; }
            {
                uint32_t v[32], pk[16];
                tmem_ld32(lane_base + kSD + h * 32, v);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) pk[i] = pack_bf16x2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
                tmem_st16(lane_base + kSA + h * 16, pk);
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    pk[i] = pack_bf16x2(__uint_as_float(v[2 * i]) - bf16_lo(pk[i]), __uint_as_float(v[2 * i + 1]) - bf16_hi(pk[i]));
                tmem_st16(lane_base + kO2 + h * 16, pk);
                tmem_wait_st();
                tc_fence_before_sync();
                handoff_arrive<4>();
            }
            // With the norms in the tables, the next chunk's tables are written after this chunk's hand-off (see above),
            // so the hand-off -> product -> completion chain does not order them before their readers: one barrier.
            if (NRM && c + 1 < n_c) asm volatile("bar.sync 1, 512;" ::: "memory");
            if (!SO && short_chunk) {
                // only the rows of real tokens leave, 16 bytes per thread and step, from the staged (swizzled) tile
                asm volatile("bar.sync 1, 512;" ::: "memory");  // (last chunk of a packed sequence only)
                for (int q = tid; q < left * 16; q += kThreads) {
                    const int tok = q >> 4, ch = q & 15;  // 16-byte piece ch of the token's 256-byte row
                    const uint4 v = *reinterpret_cast<const uint4*>(smem + kOffO + (c & 1) * kTileBytes + (ch >> 3) * 8192 +
                                                                    tok * 128 + (((ch & 7) ^ (tok & 7)) << 4));
                    *reinterpret_cast<uint4*>(p.O + (grow0 + (long long)(c * kC + tok) * gstep) * kD + ch * 8) = v;
                }
            }
        }
        if (!ok) {
            // a bounded wait ran out (s_fail is set): release the issuing and the storing warp from whichever hand-off
            // they wait on (both leave their loops when they see s_fail)
            handoff_arrive<4>();
            handoff_arrive<5>();
            handoff_arrive<6>();
        }
        // ---- final state
        if (ok && p.S_out != nullptr) {
            float* so = p.S_out + ((long long)blockIdx.x * kD + t) * kD + h * 32;
            uint32_t v[32];
            tmem_ld32(lane_base + kSD + h * 32, v);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 8; ++i)
                *reinterpret_cast<float4*>(so + i * 4) =
                    make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]), __uint_as_float(v[4 * i + 2]),
                                __uint_as_float(v[4 * i + 3]));
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0 && *fail != 0) atomicExch(p.status, GDN_ERR_TIMEOUT);
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

// [heads][T][cols] bf16 tensor (cols = 128, or H * 128 for token-major tensors with heads = B), boxes of 64 rows x 64
// columns, 128-byte swizzle
bool make_map(CUtensorMap* tm, const void* base, long long heads, int T, int cols) {
    EncodeTiledFn enc = get_encode_fn();
    if (enc == nullptr) return false;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(T), static_cast<cuuint64_t>(heads)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(cols) * 2, static_cast<cuuint64_t>(T) * cols * 2};
    cuuint32_t box[3] = {64, static_cast<cuuint32_t>(kC), 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ---- the segmented call: a long sequence cut into P segments whose state maps are formed in parallel
// Set-up of the first pass: the token ranges of its 2P - 3 runs (runs 0 .. P-2: segment s from a zero state, segment 0
// from the caller's; runs P-1 .. 2P-4: segments 1 .. P-2 from the identity with U = 0, which gives the matrix M of
// S_end = S_start M + N), their initial states, the token ranges of the second pass and its first initial state.
__global__ void segmented_setup_kernel(int P, int H_v, int n_chunks, const float* S_user, float* S_in1, float* S_start,
                                       int* start1, int* end1, int* no_u1, int* start3, int* end3) {
    const int n1 = 2 * P - 3;
    if (blockIdx.x == 0 && threadIdx.x < 32) {
        for (int s_ = threadIdx.x; s_ < n1; s_ += 32) {
            const int seg = (s_ <= P - 2) ? s_ : s_ - (P - 2);
            start1[s_] = (int)((long long)n_chunks * seg / P) * kC;
            end1[s_] = (int)((long long)n_chunks * (seg + 1) / P) * kC;
            no_u1[s_] = (s_ <= P - 2) ? 0 : 1;
        }
        for (int s_ = threadIdx.x; s_ < P; s_ += 32) {
            start3[s_] = (int)((long long)n_chunks * s_ / P) * kC;
            end3[s_] = (int)((long long)n_chunks * (s_ + 1) / P) * kC;
        }
    }
    const long long per = (long long)H_v * kD * kD;
    const long long total = (long long)n1 * per;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total + per; e += (long long)gridDim.x * blockDim.x) {
        if (e < total) {
            const int s_ = (int)(e / per);
            const long long r = e - (long long)s_ * per;
            const int idx = (int)(r % (kD * kD));
            float v = 0.f;
            if (s_ == 0) v = (S_user != nullptr) ? S_user[r] : 0.f;
            else if (s_ > P - 2) v = (idx / kD == idx % kD) ? 1.f : 0.f;
            S_in1[e] = v;
        } else {
            const long long r = e - total;
            S_start[r] = (S_user != nullptr) ? S_user[r] : 0.f;
        }
    }
}

// S_start[k] = S_start[k-1] M_{k-1} + N_{k-1} for k = 2 .. P-1, S_start[1] = N_0 (the first segment ran from the caller's
// state). One CTA per (value head, block of 16 state rows): the rows of the state are independent. fp32 FMAs.
__global__ void __launch_bounds__(256) segmented_combine_kernel(int P, int H_v, const float* S_out1, float* S_start) {
    __shared__ float cur[16][kD];
    const int hv = blockIdx.x, r0 = blockIdx.y * 16;
    const long long per = (long long)H_v * kD * kD;
    const int col = threadIdx.x & 127, rh = threadIdx.x >> 7;  // this thread: column col, rows r0 + rh, r0 + rh + 2, ...
    const float* N0 = S_out1 + (long long)hv * kD * kD;
    for (int i = 0; i < 8; ++i) {
        const int r = rh + 2 * i;
        const float v = N0[(r0 + r) * kD + col];
        cur[r][col] = v;
        S_start[per + (long long)hv * kD * kD + (r0 + r) * kD + col] = v;
    }
    __syncthreads();
    for (int k = 2; k < P; ++k) {
        const float* M = S_out1 + (long long)(P - 1 + (k - 2)) * per + (long long)hv * kD * kD;  // M of segment k - 1
        const float* N = S_out1 + (long long)(k - 1) * per + (long long)hv * kD * kD;            // N of segment k - 1
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = N[(r0 + rh + 2 * i) * kD + col];
        for (int d = 0; d < kD; ++d) {
            const float m = M[d * kD + col];
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = fmaf(cur[rh + 2 * i][d], m, acc[i]);
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            cur[rh + 2 * i][col] = acc[i];
            S_start[(long long)k * per + (long long)hv * kD * kD + (r0 + rh + 2 * i) * kD + col] = acc[i];
        }
        __syncthreads();
    }
}

}  // namespace

size_t chunk_state_segmented_workspace(int H_v, int P) {
    if (P < 2) return 0;
    const size_t per = (size_t)H_v * kD * kD * sizeof(float);
    const size_t n1 = (size_t)(2 * P - 3);
    return (2 * n1 + 2 * (size_t)P) * per + (3 * n1 + 2 * (size_t)P) * sizeof(int) + 256;
}

int chunk_state_auto_segments(long long H_v) {
    int n_sm = 0, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return 1;
    int P = 1;
    while (P < 8 && H_v * (2 * (P + 1) - 3) <= n_sm) ++P;
    return P;
}

// One sequence per value head (B = 1), cut into P segments: first pass = every segment's state map in parallel (state
// only), then the segments' initial states by a short recurrence, then every segment in parallel with its output.
int launch_chunk_state_segmented(const ProblemS& q, int P, void* workspace, cudaStream_t stream) {
    if (q.B != 1 || q.seq_start != nullptr) return GDN_ERR_UNSUPPORTED;
    const int n_chunks = q.T / kC;
    if (P > n_chunks) P = n_chunks;
    if (P < 2) return launch_chunk_state(q, stream);
    const size_t per = (size_t)q.H_v * kD * kD;
    const size_t n1 = (size_t)(2 * P - 3);
    float* S_in1 = static_cast<float*>(workspace);
    float* S_out1 = S_in1 + n1 * per;
    float* S_start = S_out1 + n1 * per;
    float* S_out3 = S_start + (size_t)P * per;
    int* start1 = reinterpret_cast<int*>(S_out3 + (size_t)P * per);
    int* end1 = start1 + n1;
    int* no_u1 = end1 + n1;
    int* start3 = no_u1 + n1;
    int* end3 = start3 + P;
    segmented_setup_kernel<<<256, 256, 0, stream>>>(P, q.H_v, n_chunks, q.S_in, S_in1, S_start, start1, end1, no_u1, start3, end3);
    count_launch();
    ProblemS a = q;
    a.B = static_cast<int>(n1);
    a.S_in = S_in1;
    a.S_out = S_out1;
    a.O = q.O;  // not written
    a.seq_start = start1;
    a.seq_end = end1;
    a.seq_no_u = no_u1;
    a.state_only = true;
    int rc = launch_chunk_state(a, stream);
    if (rc != GDN_OK) return rc;
    segmented_combine_kernel<<<dim3(q.H_v, kD / 16), 256, 0, stream>>>(P, q.H_v, S_out1, S_start);
    count_launch();
    ProblemS b = q;
    b.B = P;
    b.S_in = S_start;
    b.S_out = (q.S_out != nullptr) ? S_out3 : nullptr;
    b.seq_start = start3;
    b.seq_end = end3;
    rc = launch_chunk_state(b, stream);
    if (rc != GDN_OK) return rc;
    if (q.S_out != nullptr &&
        cudaMemcpyAsync(q.S_out, S_out3 + (size_t)(P - 1) * per, per * sizeof(float), cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
        return GDN_ERR_LAUNCH;
    return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_LAUNCH;
}

// ---- the segmented call on built-in scratch memory (for callers that cannot allocate device memory)
// The scratch lives in this file-scope device array: every GPU that loads the library holds it until the process
// exits. In host code the array's name is only a handle; the device address comes from cudaGetSymbolAddress, once per
// device, with that device current.
namespace {
constexpr size_t kBuiltinStateBlocks = 128;  // state-sized blocks of 128 x 128 fp32 (64 KB each): 8 MB
constexpr size_t kBuiltinScratchBytes = kBuiltinStateBlocks * kD * kD * sizeof(float) + 4096;
static __device__ __align__(256) unsigned char g_builtin_scratch[kBuiltinScratchBytes];
constexpr int kMaxDev = 64;
void* g_builtin_scratch_addr[kMaxDev] = {nullptr};
}  // namespace

int launch_chunk_state_segmented_builtin(const ProblemS& q, int P, cudaStream_t stream) {
    const int n_chunks = q.T / kC;
    const int p_eff = P > n_chunks ? n_chunks : P;
    if (p_eff >= 2 && chunk_state_segmented_workspace(q.H_v, p_eff) > kBuiltinScratchBytes) return GDN_ERR_SCRATCH;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return GDN_ERR_LAUNCH;
    if (g_builtin_scratch_addr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_builtin_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return GDN_ERR_LAUNCH;
        }
        g_builtin_scratch_addr[dev] = ptr;
    }
    return launch_chunk_state_segmented(q, P, g_builtin_scratch_addr[dev], stream);
}


int launch_chunk_state(const ProblemS& q, cudaStream_t stream) {
    if (q.d_k != kD || q.d_v != kD || q.C != kC) return GDN_ERR_UNSUPPORTED;
    // packed sequences: B counts the sequences, the tensors have one row of T tokens per head
    const bool var = q.seq_start != nullptr;
    if (q.state_only && !var) return GDN_ERR_UNSUPPORTED;
    const long long hk = var ? q.H_k : (long long)q.B * q.H_k, hv = var ? q.H_v : (long long)q.B * q.H_v;
    const long long n_cta = (long long)q.B * q.H_v;
    if (n_cta == 0) return GDN_OK;
    if (q.T == 0) {
        // no tokens: every sequence hands its initial state on (zeros without one)
        if (q.S_out != nullptr && !q.state_only) {
            const size_t bytes = static_cast<size_t>(n_cta) * kD * kD * sizeof(float);
            const cudaError_t e = (q.S_in != nullptr) ? cudaMemcpyAsync(q.S_out, q.S_in, bytes, cudaMemcpyDeviceToDevice, stream)
                                                      : cudaMemsetAsync(q.S_out, 0, bytes, stream);
            if (e != cudaSuccess) return GDN_ERR_LAUNCH;
        }
        return GDN_OK;
    }
    if (n_cta >= (1LL << 31)) return GDN_ERR_UNSUPPORTED;
    if (hv >= (1LL << 31)) return GDN_ERR_UNSUPPORTED;
    int* status = device_status_word();
    if (status == nullptr) return GDN_ERR_LAUNCH;
    CUtensorMap mQ, mK, mW, mU, mO;
    const bool bthd = (q.flags & GDN_FLAG_LAYOUT_BTHD) != 0;
    const long long nb = var ? 1 : q.B;
    const long long zk = bthd ? nb : hk, zv = bthd ? nb : hv;
    const int ck = bthd ? q.H_k * kD : kD, cv = bthd ? q.H_v * kD : kD;
    if (!make_map(&mQ, q.Q, zk, q.T, ck) || !make_map(&mK, q.K, zk, q.T, ck) || !make_map(&mW, q.W, zv, q.T, cv) ||
        !make_map(&mU, q.U, zv, q.T, cv) || !make_map(&mO, q.O, zv, q.T, cv))
        return GDN_ERR_LAUNCH;
    ParamsS prm;
    prm.g = q.g;
    prm.S_in = q.S_in;
    prm.S_out = q.S_out;
    prm.status = status;
    prm.H_k = q.H_k;
    prm.H_v = q.H_v;
    prm.T = q.T;
    prm.group = q.H_v / q.H_k;
    prm.scale = q.scale;
    prm.flags = q.flags;
    prm.seq_start = q.seq_start;
    prm.seq_end = q.seq_end;
    prm.seq_no_u = q.seq_no_u;
    prm.O = static_cast<__nv_bfloat16*>(q.O);
    const int smem = kSmemTotal + 1024;
    const bool nrm = (q.flags & GDN_FLAG_K_L2NORM) != 0;
    auto kern = q.state_only ? (nrm ? chunk_state_kernel<true, true, true> : chunk_state_kernel<true, true, false>)
                : var        ? (nrm ? chunk_state_kernel<true, false, true> : chunk_state_kernel<true, false, false>)
                             : (nrm ? chunk_state_kernel<false, false, true> : chunk_state_kernel<false, false, false>);
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return GDN_ERR_LAUNCH;
    kern<<<static_cast<int>(n_cta), kThreads + 64, smem, stream>>>(mQ, mK, mW, mU, mO, prm);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_LAUNCH;
}

}  // namespace gdn
