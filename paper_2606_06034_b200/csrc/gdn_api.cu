// C-ABI entry points: argument validation, kernel selection, status word.
#include <atomic>
#include <cstdint>

#include "common.cuh"

namespace gdn {

// One status word per device that loads this library; kernels write GDN_ERR_TIMEOUT here
// when a bounded wait gives up.
__device__ int g_status_word = 0;

namespace {
std::atomic<long long> g_launches{0};
constexpr int kMaxDevices = 64;
int* g_status_addr[kMaxDevices] = {nullptr};
int g_arch_ok[kMaxDevices] = {0};  // 0 unknown, 1 yes, -1 no
}  // namespace

void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

int* device_status_word() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    if (g_status_addr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_status_word) != cudaSuccess) return nullptr;
        g_status_addr[dev] = static_cast<int*>(ptr);
    }
    return g_status_addr[dev];
}

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_arch() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return GDN_ERR_ARCH;
    }
    if (g_arch_ok[dev] == 0) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
            cudaGetLastError();
            return GDN_ERR_ARCH;
        }
        g_arch_ok[dev] = (major == 10) ? 1 : -1;
    }
    return g_arch_ok[dev] == 1 ? GDN_OK : GDN_ERR_ARCH;
}

// Validation shared by every entry point. Order: NULL, sizes, alignment, architecture.
int validate(const Problem& p, bool neumann) {
    if (p.K == nullptr || p.V == nullptr || p.beta == nullptr || p.g == nullptr || p.W == nullptr || p.U == nullptr)
        return GDN_ERR_NULL;
    if (p.B < 0 || p.H_k <= 0 || p.H_v <= 0 || p.T < 0 || p.C < 2 || p.d_k <= 0 || p.d_v <= 0) return GDN_ERR_INVALID_ARG;
    if (p.H_v % p.H_k != 0) return GDN_ERR_INVALID_ARG;
    if (p.T % p.C != 0) return GDN_ERR_INVALID_ARG;
    if (p.dtype != GDN_DTYPE_FP32 && p.dtype != GDN_DTYPE_BF16) return GDN_ERR_INVALID_ARG;
    if (neumann) {
        const int blk = (p.C == 128) ? 64 : p.C;
        if (p.order < 1 || p.order >= blk || p.steps < 0) return GDN_ERR_INVALID_ARG;
    }
    if (p.C > 128) return GDN_ERR_UNSUPPORTED;
    if (p.d_k % 8 != 0 || p.d_v % 8 != 0) return GDN_ERR_UNSUPPORTED;
    if (!aligned16(p.K) || !aligned16(p.V) || !aligned16(p.beta) || !aligned16(p.g) || !aligned16(p.W) || !aligned16(p.U) ||
        !aligned16(p.Tinv))
        return GDN_ERR_ALIGN;
    return GDN_OK;
}

int run(Problem p, InverseMode mode, cudaStream_t stream) {
    const bool neumann = (mode == INV_NEUMANN);
    if (neumann) {
        if (p.order == -1) p.order = gdn_default_order(p.C);
        if (p.steps == -1) p.steps = gdn_default_residual_steps(p.C);
    }
    int rc = validate(p, neumann);
    if (rc != GDN_OK) return rc;
    rc = check_arch();
    if (rc != GDN_OK) return rc;
    if (p.dtype == GDN_DTYPE_FP32) {
        if (p.flags & GDN_FLAG_LAYOUT_BTHD) return GDN_ERR_UNSUPPORTED;  // the token-major layout is built for bf16 only
        return launch_simt(p, mode, stream);
    }
    // bf16: the tensor-core kernel is built for d_k = d_v = 128, C in {16, 32, 64, 128} and order <= 7. Other shapes
    // (any 2 <= C <= 64, feature sizes up to 256 in multiples of 8, higher orders) run on the ALU kernel with bf16
    // tensors and the same fp32 arithmetic; the token-major layout and packed sequences exist on the tensor-core
    // kernel only.
    const bool tc_shape = p.d_k == 128 && p.d_v == 128 && (p.C == 16 || p.C == 32 || p.C == 64 || p.C == 128) &&
                          (!neumann || p.order <= 7);
    if (!tc_shape) {
        if ((p.flags & GDN_FLAG_LAYOUT_BTHD) != 0 || p.chunk_start != nullptr) return GDN_ERR_UNSUPPORTED;
        return launch_simt(p, mode, stream);
    }
    return launch_tc_bf16(p, mode, stream);
}

}  // namespace
}  // namespace gdn

using namespace gdn;

extern "C" {

int gdn_chunk_prepare(const void* K, const void* V, const float* beta, const float* g, int B, int H, int T, int C, int d_k,
                      int d_v, int order, int residual_steps, int dtype, void* W_out, void* U_out, void* Tinv_out,
                      gdn_stream_t stream) {
    Problem p{K, V, beta, g, W_out, U_out, Tinv_out, B, H, H, T, C, d_k, d_v, order, residual_steps, dtype};
    return run(p, INV_NEUMANN, static_cast<cudaStream_t>(stream));
}

int gdn_chunk_prepare_gqa(const void* K, const void* V, const float* beta, const float* g, int B, int H_k, int H_v, int T, int C,
                          int d_k, int d_v, int order, int residual_steps, int dtype, void* W_out, void* U_out, void* Tinv_out,
                          gdn_stream_t stream) {
    Problem p{K, V, beta, g, W_out, U_out, Tinv_out, B, H_k, H_v, T, C, d_k, d_v, order, residual_steps, dtype};
    return run(p, INV_NEUMANN, static_cast<cudaStream_t>(stream));
}

int gdn_chunk_prepare_ex(const void* K, const void* V, const float* beta, const float* g, int B, int H_k, int H_v, int T, int C,
                         int d_k, int d_v, int order, int residual_steps, int dtype, void* W_out, void* U_out, void* Tinv_out,
                         unsigned flags, gdn_stream_t stream) {
    if (flags & ~static_cast<unsigned>(GDN_FLAG_G_RAW | GDN_FLAG_K_L2NORM | GDN_FLAG_OUT_FP32 | GDN_FLAG_LAYOUT_BTHD |
                                       GDN_FLAG_W_GATED))
        return GDN_ERR_INVALID_ARG;
    Problem p{K, V, beta, g, W_out, U_out, Tinv_out, B, H_k, H_v, T, C, d_k, d_v, order, residual_steps, dtype};
    p.flags = flags;
    return run(p, INV_NEUMANN, static_cast<cudaStream_t>(stream));
}

int gdn_chunk_prepare_varlen(const void* K, const void* V, const float* beta, const float* g, const int32_t* chunk_start,
                             const int32_t* chunk_len, int n_chunks, int T_total, int H_k, int H_v, int C, int d_k, int d_v,
                             int order, int residual_steps, void* W_out, void* U_out, void* Tinv_out, unsigned flags,
                             gdn_stream_t stream) {
    if (flags & ~static_cast<unsigned>(GDN_FLAG_G_RAW | GDN_FLAG_K_L2NORM | GDN_FLAG_LAYOUT_BTHD | GDN_FLAG_W_GATED))
        return GDN_ERR_INVALID_ARG;
    if (chunk_start == nullptr || chunk_len == nullptr) return GDN_ERR_NULL;
    if (n_chunks < 0 || T_total < 0) return GDN_ERR_INVALID_ARG;
    if (!(C == 16 || C == 32 || C == 64 || C == 128)) return C >= 2 ? GDN_ERR_UNSUPPORTED : GDN_ERR_INVALID_ARG;
    // the chunks are walked in tiles of 128 token rows: T is the padded row count
    const long long rows = ((long long)n_chunks * C + 127) / 128 * 128;
    if (rows >= (1LL << 31)) return GDN_ERR_UNSUPPORTED;
    Problem p{K, V, beta, g, W_out, U_out, Tinv_out, 1, H_k, H_v, static_cast<int>(rows), C, d_k, d_v, order, residual_steps,
              GDN_DTYPE_BF16};
    p.flags = flags;
    p.chunk_start = chunk_start;
    p.chunk_len = chunk_len;
    p.n_chunks = n_chunks;
    p.T_total = T_total;
    if (n_chunks == 0 || T_total == 0) {
        if (p.order == -1) p.order = gdn_default_order(C);
        if (p.steps == -1) p.steps = gdn_default_residual_steps(C);
        const int rc = validate(p, true);
        return rc != GDN_OK ? rc : check_arch();
    }
    return run(p, INV_NEUMANN, static_cast<cudaStream_t>(stream));
}

int gdn_chunk_prepare_fwdsubst(const void* K, const void* V, const float* beta, const float* g, int B, int H_k, int H_v, int T,
                               int C, int d_k, int d_v, int dtype, int variant, void* W_out, void* U_out, void* Tinv_out,
                               gdn_stream_t stream) {
    if (variant != GDN_FWDSUBST_ROWS && variant != GDN_FWDSUBST_BLOCKED && variant != GDN_FWDSUBST_BLOCKED_TC)
        return GDN_ERR_INVALID_ARG;
    Problem p{K, V, beta, g, W_out, U_out, Tinv_out, B, H_k, H_v, T, C, d_k, d_v, 0, 0, dtype};
    if (variant == GDN_FWDSUBST_BLOCKED_TC && (dtype != GDN_DTYPE_BF16 || C != 64)) {
        const int rc = validate(p, false);
        return rc != GDN_OK ? rc : GDN_ERR_UNSUPPORTED;
    }
    const InverseMode mode = variant == GDN_FWDSUBST_ROWS ? INV_FWDSUBST_ROWS
                             : variant == GDN_FWDSUBST_BLOCKED ? INV_FWDSUBST_BLOCKED : INV_FWDSUBST_TC;
    return run(p, mode, static_cast<cudaStream_t>(stream));
}

int gdn_chunk_prepare_int8(const int8_t* Kq, const int8_t* Vq, const int32_t* k_exp, const int32_t* v_exp, const uint16_t* beta_q,
                           const int32_t* decay_q, int B, int H_k, int H_v, int T, int C, int d_k, int d_v, int order,
                           int residual_steps, int8_t* Wq_out, int8_t* Uq_out, int32_t* w_exp_out, int32_t* u_exp_out,
                           int8_t* Toff_q_out, int32_t* t_exp_out, int32_t* dbg_acc_out, gdn_stream_t stream) {
    if (order == -1) order = gdn_default_order(C);
    if (residual_steps == -1) residual_steps = gdn_default_residual_steps(C);
    if (Kq == nullptr || Vq == nullptr || k_exp == nullptr || v_exp == nullptr || beta_q == nullptr || decay_q == nullptr ||
        Wq_out == nullptr || Uq_out == nullptr || w_exp_out == nullptr || u_exp_out == nullptr || t_exp_out == nullptr)
        return GDN_ERR_NULL;
    if (B < 0 || H_k <= 0 || H_v <= 0 || T < 0 || C < 2 || d_k <= 0 || d_v <= 0) return GDN_ERR_INVALID_ARG;
    if (H_v % H_k != 0 || T % C != 0) return GDN_ERR_INVALID_ARG;
    if (order < 1 || order >= C || residual_steps < 0) return GDN_ERR_INVALID_ARG;
    if (!aligned16(Kq) || !aligned16(Vq) || !aligned16(Wq_out) || !aligned16(Uq_out) || !aligned16(Toff_q_out) || !aligned16(dbg_acc_out))
        return GDN_ERR_ALIGN;
    const int rc = check_arch();
    if (rc != GDN_OK) return rc;
    ProblemI8 q{Kq, Vq, k_exp, v_exp, reinterpret_cast<const int16_t*>(beta_q), decay_q, Wq_out, Uq_out, w_exp_out, u_exp_out,
                Toff_q_out, t_exp_out, dbg_acc_out, B, H_k, H_v, T, C, d_k, d_v, order, residual_steps};
    return launch_tc_int8(q, static_cast<cudaStream_t>(stream));
}

int gdn_chunk_prepare_int16(const int16_t* Kq, const int16_t* Vq, const int32_t* k_exp, const int32_t* v_exp,
                            const uint16_t* beta_q, const int32_t* decay_q, int B, int H_k, int H_v, int T, int C, int d_k,
                            int d_v, int order, int residual_steps, int16_t* Wq_out, int16_t* Uq_out, int32_t* w_exp_out,
                            int32_t* u_exp_out, int16_t* Toff_q_out, int32_t* t_exp_out, int64_t* dbg_acc_out,
                            gdn_stream_t stream) {
    if (order == -1) order = gdn_default_order(C);
    if (residual_steps == -1) residual_steps = gdn_default_residual_steps(C);
    if (Kq == nullptr || Vq == nullptr || k_exp == nullptr || v_exp == nullptr || beta_q == nullptr || decay_q == nullptr ||
        Wq_out == nullptr || Uq_out == nullptr || w_exp_out == nullptr || u_exp_out == nullptr || t_exp_out == nullptr)
        return GDN_ERR_NULL;
    if (B < 0 || H_k <= 0 || H_v <= 0 || T < 0 || C < 2 || d_k <= 0 || d_v <= 0) return GDN_ERR_INVALID_ARG;
    if (H_v % H_k != 0 || T % C != 0) return GDN_ERR_INVALID_ARG;
    if (order < 1 || order >= C || residual_steps < 0) return GDN_ERR_INVALID_ARG;
    if (!aligned16(Kq) || !aligned16(Vq) || !aligned16(Wq_out) || !aligned16(Uq_out) || !aligned16(Toff_q_out) || !aligned16(dbg_acc_out))
        return GDN_ERR_ALIGN;
    const int rc = check_arch();
    if (rc != GDN_OK) return rc;
    ProblemI16 q{Kq, Vq, k_exp, v_exp, reinterpret_cast<const int16_t*>(beta_q), decay_q, Wq_out, Uq_out, w_exp_out, u_exp_out,
                 Toff_q_out, t_exp_out, reinterpret_cast<long long*>(dbg_acc_out), B, H_k, H_v, T, C, d_k, d_v, order,
                 residual_steps};
    return launch_tc_int16(q, static_cast<cudaStream_t>(stream));
}

int gdn_chunk_state_output(const void* Q, const void* K, const void* W_gated, const void* U, const float* g, int B, int H_k,
                           int H_v, int T, int C, int d_k, int d_v, float scale, const float* S_in, void* O_out, float* S_out,
                           unsigned flags, gdn_stream_t stream) {
    if (flags & ~static_cast<unsigned>(GDN_FLAG_G_RAW | GDN_FLAG_LAYOUT_BTHD | GDN_FLAG_K_L2NORM)) return GDN_ERR_INVALID_ARG;
    if (Q == nullptr || K == nullptr || W_gated == nullptr || U == nullptr || g == nullptr || O_out == nullptr) return GDN_ERR_NULL;
    if (B < 0 || H_k <= 0 || H_v <= 0 || T < 0 || C < 2 || d_k <= 0 || d_v <= 0) return GDN_ERR_INVALID_ARG;
    if (H_v % H_k != 0 || T % C != 0) return GDN_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(W_gated) || !aligned16(U) || !aligned16(g) || !aligned16(S_in) ||
        !aligned16(O_out) || !aligned16(S_out))
        return GDN_ERR_ALIGN;
    const int rc = check_arch();
    if (rc != GDN_OK) return rc;
    ProblemS q{Q, K, W_gated, U, g, S_in, O_out, S_out, B, H_k, H_v, T, C, d_k, d_v, scale, flags};
    return launch_chunk_state(q, static_cast<cudaStream_t>(stream));
}

int gdn_chunk_state_segments(int H_v) { return check_arch() == GDN_OK ? chunk_state_auto_segments(H_v) : 1; }

size_t gdn_chunk_state_segmented_workspace(int H_v, int segments) {
    return (H_v > 0 && segments >= 2) ? chunk_state_segmented_workspace(H_v, segments) : 0;
}

int gdn_chunk_state_output_segmented(const void* Q, const void* K, const void* W_gated, const void* U, const float* g, int H_k,
                                     int H_v, int T, int C, int d_k, int d_v, float scale, const float* S_in, void* O_out,
                                     float* S_out, int segments, void* workspace, size_t workspace_bytes, unsigned flags,
                                     gdn_stream_t stream) {
    if (flags & ~static_cast<unsigned>(GDN_FLAG_G_RAW | GDN_FLAG_LAYOUT_BTHD | GDN_FLAG_K_L2NORM)) return GDN_ERR_INVALID_ARG;
    if (Q == nullptr || K == nullptr || W_gated == nullptr || U == nullptr || g == nullptr || O_out == nullptr) return GDN_ERR_NULL;
    if (H_k <= 0 || H_v <= 0 || T < 0 || C < 2 || d_k <= 0 || d_v <= 0 || segments < 1 || segments > 64) return GDN_ERR_INVALID_ARG;
    if (H_v % H_k != 0 || T % C != 0) return GDN_ERR_INVALID_ARG;
    if (segments >= 2 && workspace == nullptr) return GDN_ERR_NULL;
    if (segments >= 2 && workspace_bytes < chunk_state_segmented_workspace(H_v, segments)) return GDN_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(W_gated) || !aligned16(U) || !aligned16(g) || !aligned16(S_in) ||
        !aligned16(O_out) || !aligned16(S_out) || !aligned16(workspace))
        return GDN_ERR_ALIGN;
    const int rc = check_arch();
    if (rc != GDN_OK) return rc;
    ProblemS q{Q, K, W_gated, U, g, S_in, O_out, S_out, 1, H_k, H_v, T, C, d_k, d_v, scale, flags};
    return launch_chunk_state_segmented(q, segments, workspace, static_cast<cudaStream_t>(stream));
}

int gdn_chunk_state_output_segmented_noalloc(const void* Q, const void* K, const void* W_gated, const void* U, const float* g,
                                             int H_k, int H_v, int T, int C, int d_k, int d_v, float scale, const float* S_in,
                                             void* O_out, float* S_out, int segments, unsigned flags, gdn_stream_t stream) {
    if (flags & ~static_cast<unsigned>(GDN_FLAG_G_RAW | GDN_FLAG_LAYOUT_BTHD | GDN_FLAG_K_L2NORM)) return GDN_ERR_INVALID_ARG;
    if (Q == nullptr || K == nullptr || W_gated == nullptr || U == nullptr || g == nullptr || O_out == nullptr) return GDN_ERR_NULL;
    if (H_k <= 0 || H_v <= 0 || T < 0 || C < 2 || d_k <= 0 || d_v <= 0 || segments < 1 || segments > 64) return GDN_ERR_INVALID_ARG;
    if (H_v % H_k != 0 || T % C != 0) return GDN_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(W_gated) || !aligned16(U) || !aligned16(g) || !aligned16(S_in) ||
        !aligned16(O_out) || !aligned16(S_out))
        return GDN_ERR_ALIGN;
    const int rc = check_arch();
    if (rc != GDN_OK) return rc;
    ProblemS q{Q, K, W_gated, U, g, S_in, O_out, S_out, 1, H_k, H_v, T, C, d_k, d_v, scale, flags};
    return launch_chunk_state_segmented_builtin(q, segments, static_cast<cudaStream_t>(stream));
}

int gdn_chunk_state_output_varlen(const void* Q, const void* K, const void* W_gated, const void* U, const float* g,
                                  const int32_t* cu_seqlens, int n_seq, int T_total, int H_k, int H_v, int C, int d_k, int d_v,
                                  float scale, const float* S_in, void* O_out, float* S_out, unsigned flags,
                                  gdn_stream_t stream) {
    if (flags & ~static_cast<unsigned>(GDN_FLAG_G_RAW | GDN_FLAG_LAYOUT_BTHD | GDN_FLAG_K_L2NORM)) return GDN_ERR_INVALID_ARG;
    if (Q == nullptr || K == nullptr || W_gated == nullptr || U == nullptr || g == nullptr || O_out == nullptr ||
        cu_seqlens == nullptr)
        return GDN_ERR_NULL;
    if (n_seq < 0 || H_k <= 0 || H_v <= 0 || T_total < 0 || C < 2 || d_k <= 0 || d_v <= 0) return GDN_ERR_INVALID_ARG;
    if (H_v % H_k != 0) return GDN_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(W_gated) || !aligned16(U) || !aligned16(g) || !aligned16(S_in) ||
        !aligned16(O_out) || !aligned16(S_out))
        return GDN_ERR_ALIGN;
    const int rc = check_arch();
    if (rc != GDN_OK) return rc;
    ProblemS q{Q, K, W_gated, U, g, S_in, O_out, S_out, n_seq, H_k, H_v, T_total, C, d_k, d_v, scale, flags};
    q.seq_start = cu_seqlens;
    q.seq_end = cu_seqlens + 1;
    return launch_chunk_state(q, static_cast<cudaStream_t>(stream));
}

int gdn_selftest_bounded_wait(gdn_stream_t stream) {
    const int rc = check_arch();
    if (rc != GDN_OK) return rc;
    return launch_wait_selftest(static_cast<cudaStream_t>(stream));
}

unsigned int gdn_int8_lut_checksum(void) {
    uint16_t lut[256];
    int8_decay_lut(lut);
    unsigned long long s = 0;
    for (int f = 0; f < 256; ++f) s = (s * 31 + lut[f] + f) % 1000000007ull;
    return static_cast<unsigned int>(s);
}

int gdn_device_status(gdn_stream_t stream) {
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        cudaGetLastError();
        return GDN_ERR_LAUNCH;
    }
    int* addr = device_status_word();
    if (addr == nullptr) return GDN_ERR_LAUNCH;
    int value = 0;
    if (cudaMemcpy(&value, addr, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return GDN_ERR_LAUNCH;
    if (value != 0) {
        const int zero = 0;
        if (cudaMemcpy(addr, &zero, sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) return GDN_ERR_LAUNCH;
    }
    return value;
}

int gdn_default_order(int C) {
    return C > 3 ? 3 : (C > 1 ? C - 1 : 1);  // (the order must stay below the chunk size: C = 2, 3 get C - 1, which is exact)
}

int gdn_default_residual_steps(int C) {
    switch (C) {
        case 16: return 3;
        case 32: return 4;
        case 64: return 8;
        case 128: return 8;
        default: {
            const int s = (C + 3) / 4 - 1;
            return s < 0 ? 0 : s;
        }
    }
}

const char* gdn_status_string(int status) {
    switch (status) {
        case GDN_OK: return "ok";
        case GDN_ERR_INVALID_ARG: return "invalid argument";
        case GDN_ERR_UNSUPPORTED: return "unsupported configuration";
        case GDN_ERR_NULL: return "null pointer";
        case GDN_ERR_ALIGN: return "pointer not 16-byte aligned";
        case GDN_ERR_LAUNCH: return "CUDA launch or set-up failed";
        case GDN_ERR_TIMEOUT: return "bounded wait inside a kernel ran out";
        case GDN_ERR_ARCH: return "device is not sm_100";
        case GDN_ERR_SCRATCH: return "problem needs more scratch memory than the library's built-in array holds";
        default: return "unknown status";
    }
}

long long gdn_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
