// Plain-FMA (no tensor core) kernel for the chunk-prepare path: one CTA per chunk,
// every matrix of the chunk in shared memory, fp32 arithmetic throughout.
//
// It serves the fp32 configuration (tolerance 1e-5 against the fp64 definition), small and
// odd chunk sizes, and the row-sequential forward-substitution comparison (Eq. 2-3). It follows
// Alg. 1 step by step with dense products: T0 = mask(sum_{n<=N} Abar^n), E = I - (I - Abar) T0,
// T = T0 * sum_{s<=S} E^s, and App. E's two-block formula for C = 128.
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

// Inverse of (I - Abar) for one n x n diagonal block by the paper's scheme (Alg. 1, right product).
// X: Abar block (ld = ldx); result written to Tout (ld = ldt). w0..w2: n x n work matrices (ld = ldw).
__device__ void neumann_block(const float* X, int ldx, float* Tout, int ldt, float* w0, float* w1, float* w2, int ldw, int n, int N,
                              int S) {
    float* T0 = w0;
    float* P = w1;
    float* Q = w2;
    // T0 = I + Abar, P = Abar
    for (int idx = threadIdx.x; idx < n * n; idx += kThreads) {
        const int i = idx / n, j = idx % n;
        const float a = X[i * ldx + j];
        P[i * ldw + j] = a;
        T0[i * ldw + j] = a + (i == j ? 1.f : 0.f);
    }
    __syncthreads();
    for (int p = 2; p <= N; ++p) {  // P <- P * Abar; T0 += P
        for (int idx = threadIdx.x; idx < n * n; idx += kThreads) {
            const int i = idx / n, j = idx % n;
            float acc = 0.f;
            for (int k = 0; k < n; ++k) acc = fmaf(P[i * ldw + k], X[k * ldx + j], acc);
            Q[i * ldw + j] = acc;
        }
        __syncthreads();
        for (int idx = threadIdx.x; idx < n * n; idx += kThreads) {
            const int i = idx / n, j = idx % n;
            T0[i * ldw + j] += Q[i * ldw + j];
        }
        float* t = P; P = Q; Q = t;
        __syncthreads();
    }
    // band mask 0 <= i - j <= N (Eq. 10)
    for (int idx = threadIdx.x; idx < n * n; idx += kThreads) {
        const int i = idx / n, j = idx % n;
        if (i - j < 0 || i - j > N) T0[i * ldw + j] = 0.f;
    }
    __syncthreads();
    // E = I - (I - Abar) T0 = I - T0 + Abar T0   -> into P ; running power in Q ; sum in Tout
    for (int idx = threadIdx.x; idx < n * n; idx += kThreads) {
        const int i = idx / n, j = idx % n;
        float acc = 0.f;
        for (int k = 0; k < n; ++k) acc = fmaf(X[i * ldx + k], T0[k * ldw + j], acc);
        const float e = (i == j ? 1.f : 0.f) - T0[i * ldw + j] + acc;
        P[i * ldw + j] = e;
    }
    __syncthreads();
    // power sum: Sum = I + E + ... + E^S, kept in Tout; running power R
    // R lives in Q and a temporary in Tout is not possible, so use registers per element:
    for (int idx = threadIdx.x; idx < n * n; idx += kThreads) {
        const int i = idx / n, j = idx % n;
        const float e = (S >= 1) ? P[i * ldw + j] : 0.f;
        Q[i * ldw + j] = e;                               // R = E
        Tout[i * ldt + j] = e + (i == j ? 1.f : 0.f);     // Sum = I + E
    }
    __syncthreads();
    for (int s = 2; s <= S; ++s) {  // R <- R * E (in place needs a temp: compute rows to registers)
        // each thread computes its elements from the old R, then all write after a barrier
        float tmp[16];  // n <= 64: at most 64 * 64 / 256 elements per thread
        int cnt = 0;
        for (int idx = threadIdx.x; idx < n * n; idx += kThreads) {
            const int i = idx / n, j = idx % n;
            float acc = 0.f;
            for (int k = 0; k < n; ++k) acc = fmaf(Q[i * ldw + k], P[k * ldw + j], acc);
            tmp[cnt++] = acc;
        }
        __syncthreads();
        cnt = 0;
        for (int idx = threadIdx.x; idx < n * n; idx += kThreads) {
            const int i = idx / n, j = idx % n;
            const float v = tmp[cnt++];
            Q[i * ldw + j] = v;
            Tout[i * ldt + j] += v;
        }
        __syncthreads();
    }
    // T = T0 * Sum  (Sum in Tout) -> needs a temp: P is free now (E no longer needed)
    for (int idx = threadIdx.x; idx < n * n; idx += kThreads) {
        const int i = idx / n, j = idx % n;
        float acc = 0.f;
        for (int k = 0; k < n; ++k) acc = fmaf(T0[i * ldw + k], Tout[k * ldt + j], acc);
        P[i * ldw + j] = acc;
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < n * n; idx += kThreads) {
        const int i = idx / n, j = idx % n;
        Tout[i * ldt + j] = P[i * ldw + j];
    }
    __syncthreads();
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
            float rn = 1.f;
            if (flags & GDN_FLAG_K_L2NORM) {
                float ss = 0.f;
                for (int d = 0; d < d_k; ++d) {
                    const float k = to_f32<IO>(Kc + (long long)i * d_k + d);
                    ss = fmaf(k, k, ss);
                }
                rn = rsqrtf(fmaxf(ss, 1e-30f));
            }
            srn[i] = rn;
        }
        __syncthreads();
        if ((flags & GDN_FLAG_G_RAW) && threadIdx.x == 0) {
            // raw log-gates: chunk-local inclusive prefix sum
            for (int i = 1; i < C; ++i) sg[i] += sg[i - 1];
        }
        __syncthreads();
        // Abar = -tril(diag(beta) (K K^T o Gamma), -1)
        for (int idx = threadIdx.x; idx < C * C; idx += kThreads) {
            const int i = idx / C, j = idx % C;
            float a = 0.f;
            if (i > j) {
                float dot = 0.f;
                for (int d = 0; d < d_k; ++d) dot = fmaf(to_f32<IO>(Kc + (long long)i * d_k + d), to_f32<IO>(Kc + (long long)j * d_k + d), dot);
                a = -sbeta[i] * expf(sg[i] - sg[j]) * dot * srn[i] * srn[j];
            }
            sA[i * ld + j] = a;
            sT[i * ld + j] = 0.f;
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
            for (int j = 0; j <= i; ++j)
                acc = fmaf(sT[i * ld + j] * sbeta[j] * srn[j] * ((flags & GDN_FLAG_W_GATED) ? expf(sg[j]) : 1.f),
                           to_f32<IO>(Kc + (long long)j * d_k + d), acc);
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
    const size_t smem = sizeof(float) * (2 * (size_t)C * (C + 1) + 3 * (size_t)blk * (blk + 1) + 3 * (size_t)C);
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
