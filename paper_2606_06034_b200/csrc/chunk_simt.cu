// Plain-FMA (no tensor core) kernel for the chunk-prepare path: one CTA per chunk,
// every matrix of the chunk in shared memory, fp32 arithmetic throughout.
//
// It serves the fp32 configuration (tolerance 1e-5 against the fp64 definition), small and
// odd chunk sizes, and the forward-substitution comparisons (Eq. 2-3, App. E). The scheme of
// Sec. 3 is evaluated through its structure rather than as dense products:
//   * the band L = T0 - I (1 <= i-j <= N) by the distance recursion
//       L_d[i] = Abar[i][i-d] + sum_{e<d} Abar[i][i-e] L_{d-e}[i-e],
//     which equals the band of sum_{n<=N} Abar^n (a band entry at distance d only receives powers n <= d);
//   * E = Abar + Abar L on i-j > N (Eq. 13 with T0 = I + L; exactly zero inside the band), N multiply-adds per entry;
//   * X_0 = T0, X_{k+1} = T0 + X_k E for k < S (so X_S = T0 sum_{s<=S} E^s), every product summed over
//     j+N+1 <= k <= i only (X is lower triangular, E vanishes for k-j <= N);
//   * App. E's two-block formula for C = 128.
// The Gram matrix is accumulated from slices of K staged in shared memory.
#include "common.cuh"

namespace gdn {
namespace {

template <typename T>
__device__ __forceinline__ float to_f32(const T* p);
template <>
__device__ __forceinline__ float to_f32<float>(const float* p) { return *p; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void st(float* p, float v) { *p = v; }
__device__ __forceinline__ void st(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

constexpr int kThreads = 256;
constexpr int kSlice = 32;  // features of K staged per step of the Gram accumulation

// Inverse of (I - Abar) for one n x n diagonal block by the truncated scheme (order N, S residual terms).
// X: Abar block (ld = ldx, strictly lower triangular); result written to Tout (ld = ldt).
// w0..w2: n x n work matrices (ld = ldw).
__device__ void neumann_block(const float* X, int ldx, float* Tout, int ldt, float* w0, float* w1, float* w2, int ldw, int n, int N,
                              int S) {
    float* T0 = w0;  // I + L, zero outside the band
    float* E = w1;
    float* Y = w2;   // second buffer of the rounds
    for (int idx = threadIdx.x; idx < n * n; idx += kThreads) {
        const int i = idx / n, j = idx % n;
        T0[i * ldw + j] = (i == j) ? 1.f : 0.f;
    }
    __syncthreads();
    // band by distance: one row per thread, one barrier per distance (row i needs L_{d-e} of rows i-e)
    for (int d = 1; d <= N && d < n; ++d) {
        for (int i = d + threadIdx.x; i < n; i += kThreads) {
            float acc = X[i * ldx + (i - d)];
            for (int e = 1; e < d; ++e) acc = fmaf(X[i * ldx + (i - e)], T0[(i - e) * ldw + (i - d)], acc);
            T0[i * ldw + (i - d)] = acc;
        }
        __syncthreads();
    }
    // E on i - j > N: Abar[i][j] + sum_{e=1..N} Abar[i][j+e] L[j+e][j]   (j + e < i always holds there)
    for (int idx = threadIdx.x; idx < n * n; idx += kThreads) {
        const int i = idx / n, j = idx % n;
        float e_ij = 0.f;
        if (i - j > N) {
            e_ij = X[i * ldx + j];
            for (int e = 1; e <= N; ++e) e_ij = fmaf(X[i * ldx + j + e], T0[(j + e) * ldw + j], e_ij);
        }
        E[i * ldw + j] = e_ij;
        Tout[i * ldt + j] = T0[i * ldw + j];  // X_0 = T0
    }
    __syncthreads();
    // X_{k+1} = T0 + X_k E: only entries with i - j > N change; the sum runs over j + N + 1 <= k <= i
    float* cur = Tout;
    int ldc = ldt;
    float* nxt = Y;
    int ldn = ldw;
    for (int r = 0; r < S; ++r) {
        for (int idx = threadIdx.x; idx < n * n; idx += kThreads) {
            const int i = idx / n, j = idx % n;
            float acc = T0[i * ldw + j];
            for (int k = j + N + 1; k <= i; ++k) acc = fmaf(cur[i * ldc + k], E[k * ldw + j], acc);
            nxt[i * ldn + j] = acc;
        }
        __syncthreads();
        float* tp = cur; cur = nxt; nxt = tp;
        const int tl = ldc; ldc = ldn; ldn = tl;
    }
    if (cur != Tout) {
        for (int idx = threadIdx.x; idx < n * n; idx += kThreads) {
            const int i = idx / n, j = idx % n;
            Tout[i * ldt + j] = cur[i * ldc + j];
        }
        __syncthreads();
    }
}

template <typename IO>
__global__ void __launch_bounds__(kThreads) chunk_simt_kernel(const IO* __restrict__ K, const IO* __restrict__ V,
                                                             const float* __restrict__ beta, const float* __restrict__ g,
                                                             IO* __restrict__ W, IO* __restrict__ U, IO* __restrict__ Tinv, int H_k,
                                                             int H_v, int T, int C, int d_k, int d_v, int N, int S, int mode,
                                                             long long n_chunks, unsigned flags) {
    extern __shared__ float sm[];
    const int ld = C + 1;
    const int blk = (C == 128) ? 64 : C;  // size of the diagonal blocks inverted by the series
    const int ldw = blk + 1;
    float* sA = sm;                 // Abar, C x C
    float* sT = sA + C * ld;        // T, C x C
    float* w0 = sT + C * ld;        // three blk x blk work matrices
    float* w1 = w0 + blk * ldw;
    float* w2 = w1 + blk * ldw;
    float* sbeta = w2 + blk * ldw;  // C
    float* sg = sbeta + C;          // C
    float* srn = sg + C;            // C: 1 / ||K_row|| (1 unless the keys are normalised here)
    float* swsc = srn + C;          // C: column scale of the W operand (beta / ||K||, times exp(g) for the gated W)
    float* sKs = swsc + C;          // C x (kSlice + 1): slice of K while the Gram matrix is accumulated
    __shared__ float swt[kThreads / 32];

    const int n_c = T / C;
    const int group = H_v / H_k;
    for (long long chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x) {
        const long long bh = chunk / n_c;
        const int c = static_cast<int>(chunk % n_c);
        const long long b = bh / H_v;
        const int hv = static_cast<int>(bh % H_v);
        const int hk = hv / group;
        const IO* Kc = K + ((b * H_k + hk) * (long long)T + (long long)c * C) * d_k;
        const IO* Vc = V + (bh * (long long)T + (long long)c * C) * d_v;
        const float* bc = beta + bh * (long long)T + (long long)c * C;
        const float* gc = g + bh * (long long)T + (long long)c * C;
        IO* Wc = W + (bh * (long long)T + (long long)c * C) * d_k;
        IO* Uc = U + (bh * (long long)T + (long long)c * C) * d_v;

        for (int i = threadIdx.x; i < C; i += kThreads) {
            sbeta[i] = bc[i];
            sg[i] = gc[i];
            srn[i] = 0.f;  // (sum of squares first)
        }
        for (int idx = threadIdx.x; idx < C * C; idx += kThreads) {
            sA[(idx / C) * ld + (idx % C)] = 0.f;
            sT[(idx / C) * ld + (idx % C)] = 0.f;
        }
        __syncthreads();
        if (flags & GDN_FLAG_G_RAW) {
            // raw log-gates: chunk-local inclusive prefix sum (C <= 128 <= kThreads): shuffles inside a warp, then the
            // totals of the warps before it
            const int i = threadIdx.x, lane = i & 31, wp = i >> 5;
            float v = (i < C) ? sg[i] : 0.f;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const float u = __shfl_up_sync(0xFFFFFFFFu, v, off);
                if (lane >= off) v += u;
            }
            if (lane == 31) swt[wp] = v;
            __syncthreads();
            for (int w = 0; w < wp; ++w) v += swt[w];
            if (i < C) sg[i] = v;
            __syncthreads();
        }
        // Gram matrix of the chunk's keys, lower triangle, from slices of kSlice features staged in shared memory
        // (every element of K is read from global memory once); the diagonal gives the row norms
        for (int d0 = 0; d0 < d_k; d0 += kSlice) {
            const int dw = min(kSlice, d_k - d0);
            for (int idx = threadIdx.x; idx < C * dw; idx += kThreads) {
                const int i = idx / dw, d = idx % dw;
                sKs[i * (kSlice + 1) + d] = to_f32<IO>(Kc + (long long)i * d_k + d0 + d);
            }
            __syncthreads();
            for (int idx = threadIdx.x; idx < C * C; idx += kThreads) {
                const int i = idx / C, j = idx % C;
                if (j > i) continue;
                float dot = 0.f;
                for (int d = 0; d < dw; ++d) dot = fmaf(sKs[i * (kSlice + 1) + d], sKs[j * (kSlice + 1) + d], dot);
                if (i == j) srn[i] += dot;
                else sA[i * ld + j] += dot;
            }
            __syncthreads();
        }
        for (int i = threadIdx.x; i < C; i += kThreads) {
            const float rn = (flags & GDN_FLAG_K_L2NORM) ? rsqrtf(fmaxf(srn[i], 1e-30f)) : 1.f;
            srn[i] = rn;
            swsc[i] = sbeta[i] * rn * ((flags & GDN_FLAG_W_GATED) ? expf(sg[i]) : 1.f);
        }
        __syncthreads();
        // Abar = -tril(diag(beta) (K K^T o Gamma), -1)
        for (int idx = threadIdx.x; idx < C * C; idx += kThreads) {
            const int i = idx / C, j = idx % C;
            if (i > j) sA[i * ld + j] = -sbeta[i] * expf(sg[i] - sg[j]) * sA[i * ld + j] * srn[i] * srn[j];
        }
        __syncthreads();

        if (mode == INV_NEUMANN) {
            const int nb = C / blk;
            for (int bi = 0; bi < nb; ++bi) {
                neumann_block(sA + bi * blk * ld + bi * blk, ld, sT + bi * blk * ld + bi * blk, ld, w0, w1, w2, ldw, blk, N, S);
            }
            if (nb == 2) {
                // Y = A21 T11 (A21 = -Abar21);  T21 = -T22 Y   (App. E, Eq. 28)
                const float* A21 = sA + blk * ld;
                const float* T11 = sT;
                const float* T22 = sT + blk * ld + blk;
                for (int idx = threadIdx.x; idx < blk * blk; idx += kThreads) {
                    const int i = idx / blk, j = idx % blk;
                    float acc = 0.f;
                    for (int k = 0; k < blk; ++k) acc = fmaf(-A21[i * ld + k], T11[k * ld + j], acc);
                    w0[i * ldw + j] = acc;
                }
                __syncthreads();
                for (int idx = threadIdx.x; idx < blk * blk; idx += kThreads) {
                    const int i = idx / blk, j = idx % blk;
                    float acc = 0.f;
                    for (int k = 0; k < blk; ++k) acc = fmaf(T22[i * ld + k], w0[k * ldw + j], acc);
                    sT[(blk + i) * ld + j] = -acc;
                }
                __syncthreads();
            }
        } else if (mode == INV_FWDSUBST_BLOCKED) {
            // Blocked form (App. E): 16 x 16 diagonal blocks by substitution (Eq. 25), then block rows from
            // S_ij = S_ii sum_{k<i} Abar_ik S_kj (Eq. 27 with T_ik = -Abar_ik); thread j owns column j.
            for (int j = threadIdx.x; j < C; j += kThreads) {
                const int bend = (j / 16 + 1) * 16;
                for (int i = j + 1; i < bend; ++i) {
                    float acc = sA[i * ld + j];
                    for (int k = j + 1; k < i; ++k) acc = fmaf(sA[i * ld + k], sT[k * ld + j], acc);
                    sT[i * ld + j] = acc;
                }
                sT[j * ld + j] = 1.f;
            }
            __syncthreads();
            for (int j = threadIdx.x; j < C; j += kThreads) {
                for (int bi = j / 16 + 1; bi < C / 16; ++bi) {
                    float tmp[16];
                    for (int r = 0; r < 16; ++r) {
                        float acc = 0.f;
                        for (int k = j; k < bi * 16; ++k) acc = fmaf(sA[(bi * 16 + r) * ld + k], sT[k * ld + j], acc);
                        tmp[r] = acc;
                    }
                    for (int r = 0; r < 16; ++r) {
                        float acc = 0.f;
                        for (int q = 0; q <= r; ++q) acc = fmaf(sT[(bi * 16 + r) * ld + bi * 16 + q], tmp[q], acc);
                        sT[(bi * 16 + r) * ld + j] = acc;
                    }
                }
            }
            __syncthreads();
        } else {
            // Forward substitution (Eq. 2-3): row i of X = Abar_i + Abar_{i,0:i} X_{0:i,:}; thread j owns column j.
            for (int j = threadIdx.x; j < C; j += kThreads) {
                for (int i = j + 1; i < C; ++i) {
                    float acc = sA[i * ld + j];
                    for (int k = j + 1; k < i; ++k) acc = fmaf(sA[i * ld + k], sT[k * ld + j], acc);
                    sT[i * ld + j] = acc;
                }
                sT[j * ld + j] = 1.f;  // Eq. 3
            }
            __syncthreads();
        }

        // W = T diag(beta) K, U = T diag(beta) V; T is lower triangular
        for (int idx = threadIdx.x; idx < C * d_k; idx += kThreads) {
            const int i = idx / d_k, d = idx % d_k;
            float acc = 0.f;
            for (int j = 0; j <= i; ++j) acc = fmaf(sT[i * ld + j] * swsc[j], to_f32<IO>(Kc + (long long)j * d_k + d), acc);
            st(Wc + (long long)i * d_k + d, acc);
        }
        for (int idx = threadIdx.x; idx < C * d_v; idx += kThreads) {
            const int i = idx / d_v, d = idx % d_v;
            float acc = 0.f;
            for (int j = 0; j <= i; ++j) acc = fmaf(sT[i * ld + j] * sbeta[j], to_f32<IO>(Vc + (long long)j * d_v + d), acc);
            st(Uc + (long long)i * d_v + d, acc);
        }
        if (Tinv != nullptr) {
            IO* Tc = Tinv + chunk * (long long)C * C;
            for (int idx = threadIdx.x; idx < C * C; idx += kThreads) st(Tc + idx, sT[(idx / C) * ld + (idx % C)]);
        }
        __syncthreads();
    }
}

}  // namespace

int launch_simt(const Problem& p, InverseMode mode, cudaStream_t stream) {
    const int C = p.C;
    if (!(C >= 2 && (C <= 64 || C == 128))) return GDN_ERR_UNSUPPORTED;
    if (p.d_k > 256 || p.d_v > 256) return GDN_ERR_UNSUPPORTED;
    if (mode == INV_FWDSUBST_BLOCKED && C % 16 != 0) return GDN_ERR_UNSUPPORTED;
    if (p.flags & GDN_FLAG_OUT_FP32) {
        if (p.dtype != GDN_DTYPE_FP32) return GDN_ERR_UNSUPPORTED;  // this kernel writes the element type it reads
    }
    const long long n_chunks = (long long)p.B * p.H_v * (p.T / C);
    if (n_chunks == 0) return GDN_OK;
    const int blk = (C == 128) ? 64 : C;
    const size_t smem = sizeof(float) * (2 * (size_t)C * (C + 1) + 3 * (size_t)blk * (blk + 1) + 4 * (size_t)C +
                                         (size_t)C * (kSlice + 1));
    const int grid = (int)(n_chunks < 148LL * 8 ? n_chunks : 148LL * 8);
    cudaError_t e;
    if (p.dtype == GDN_DTYPE_FP32) {
        e = cudaFuncSetAttribute(chunk_simt_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return GDN_ERR_LAUNCH;
        chunk_simt_kernel<float><<<grid, kThreads, smem, stream>>>((const float*)p.K, (const float*)p.V, p.beta, p.g, (float*)p.W,
                                                                  (float*)p.U, (float*)p.Tinv, p.H_k, p.H_v, p.T, C, p.d_k, p.d_v,
                                                                  p.order, p.steps, (int)mode, n_chunks, p.flags);
    } else {
        e = cudaFuncSetAttribute(chunk_simt_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return GDN_ERR_LAUNCH;
        chunk_simt_kernel<__nv_bfloat16><<<grid, kThreads, smem, stream>>>(
            (const __nv_bfloat16*)p.K, (const __nv_bfloat16*)p.V, p.beta, p.g, (__nv_bfloat16*)p.W, (__nv_bfloat16*)p.U,
            (__nv_bfloat16*)p.Tinv, p.H_k, p.H_v, p.T, C, p.d_k, p.d_v, p.order, p.steps, (int)mode, n_chunks, p.flags);
    }
    count_launch();
    return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_LAUNCH;
}

}  // namespace gdn
