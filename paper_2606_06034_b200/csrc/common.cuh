// Shared declarations of the library's translation units (host side).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>
#include <cuda_bf16.h>

#include "../../include/gdnprep.h"

namespace gdn {

// Problem description shared by all kernels.
struct Problem {
    const void* K;
    const void* V;
    const float* beta;
    const float* g;
    void* W;
    void* U;
    void* Tinv;  // may be null
    int B, H_k, H_v, T, C, d_k, d_v;
    int order;   // N
    int steps;   // S
    int dtype;   // GDN_DTYPE_*
    unsigned flags = 0;  // GDN_FLAG_*
    // packed variable-length sequences (B = 1): device arrays with the first token and the length of every chunk;
    // T is then the padded token count (a multiple of 128), T_total the number of tokens the tensors hold
    const int* chunk_start = nullptr;
    const int* chunk_len = nullptr;
    int n_chunks = 0;
    int T_total = 0;
};

// INT8 entry point's problem description
struct ProblemI8 {
    const int8_t* Kq;
    const int8_t* Vq;
    const int32_t* k_exp;
    const int32_t* v_exp;
    const int16_t* beta_q;
    const int32_t* decay_q;
    int8_t* Wq;
    int8_t* Uq;
    int32_t* w_exp;
    int32_t* u_exp;
    int8_t* Toff;  // may be null
    int32_t* t_exp;
    int32_t* dbg;  // may be null: tensor-core accumulators of the chain
    int B, H_k, H_v, T, C, d_k, d_v;
    int order, steps;
};

// INT16 entry point's problem description (the INT8 one with 16-bit mantissas and 64-bit debug accumulators)
struct ProblemI16 {
    const int16_t* Kq;
    const int16_t* Vq;
    const int32_t* k_exp;
    const int32_t* v_exp;
    const int16_t* beta_q;
    const int32_t* decay_q;
    int16_t* Wq;
    int16_t* Uq;
    int32_t* w_exp;
    int32_t* u_exp;
    int16_t* Toff;  // may be null
    int32_t* t_exp;
    long long* dbg;  // may be null: exact matrix products of the chain
    int B, H_k, H_v, T, C, d_k, d_v;
    int order, steps;
};

// State passing + output of the layer, given W (gated) and U of every chunk
struct ProblemS {
    const void* Q;
    const void* K;
    const void* W;
    const void* U;
    const float* g;
    const float* S_in;  // may be null (zero state)
    void* O;
    float* S_out;       // may be null
    int B, H_k, H_v, T, C, d_k, d_v;
    float scale;
    unsigned flags;
    // packed variable-length sequences: B sequences, sequence s = tokens [seq_start[s], seq_end[s]) of tensors with T
    // tokens per head (device arrays of B int32; the public call passes cu_seqlens and cu_seqlens + 1); null for dense
    const int* seq_start = nullptr;
    const int* seq_end = nullptr;
    // state only (packed form): no queries, no output, only S_out; seq_no_u[s] != 0: sequence s runs with U = 0
    bool state_only = false;
    const int* seq_no_u = nullptr;
};

enum InverseMode { INV_NEUMANN = 0, INV_FWDSUBST_ROWS = 1, INV_FWDSUBST_BLOCKED = 2, INV_FWDSUBST_TC = 3 };

// Status word written by kernels (one per device, static device memory).
int* device_status_word();  // device address for the current device (nullptr on failure)
void count_launch();

// Kernel launchers. Each returns a gdn_status and launches on `stream`.
int launch_simt(const Problem& p, InverseMode mode, cudaStream_t stream);
int launch_tc_bf16(const Problem& p, InverseMode mode, cudaStream_t stream);
int launch_wait_selftest(cudaStream_t stream);
int launch_chunk_state(const ProblemS& p, cudaStream_t stream);
// the segmented form for few long sequences (B = 1): P segments per sequence, workspace of chunk_state_segmented_workspace bytes
int launch_chunk_state_segmented(const ProblemS& q, int P, void* workspace, cudaStream_t stream);
size_t chunk_state_segmented_workspace(int H_v, int P);
// the same on the library's built-in scratch array (GDN_ERR_SCRATCH when the problem needs more than it holds)
int launch_chunk_state_segmented_builtin(const ProblemS& q, int P, cudaStream_t stream);
int chunk_state_auto_segments(long long H_v);
int launch_tc_int8(const ProblemI8& p, cudaStream_t stream);
int launch_tc_int16(const ProblemI16& p, cudaStream_t stream);
void int8_decay_lut(uint16_t* out256);  // table of round(2^15 * 2^(-f/256))

}  // namespace gdn
