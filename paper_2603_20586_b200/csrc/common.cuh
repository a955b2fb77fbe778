// Internal declarations shared by the kernels of the FastMKA library (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "mka.h"

namespace mka {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kTileM = 128;   // query rows per tile of the tensor-core forward
constexpr int kTileN = 128;   // key rows per tile

// Layout of the caller's workspace: a 256-byte header (device status word first), then the
// per-entry-point scratch.
constexpr size_t kWsHeader = 256;

struct LevelDev {
    const void* k;
    const void* v;
    long long n, sb, sh, sn;
};

struct LevelGradDev {
    void* dk;
    void* dv;
    long long n, sb, sh, sn;
};

struct PagedLevelDev;
struct FwdParams {
    const void* Q;
    void* O;
    float* LSE;         // may be null
    const float* gate;  // [B,T,3]
    LevelDev L[3];
    int B, H, T, d;
    int window, q_offset;
    float scale;        // tau
    int mode;
    int decode;         // every row visible
    int kv_group;       // query heads per KV head (>= 1): head h reads KV head h / kv_group
    int test_stall;     // MKA_FLAG_TEST_STALL (tensor-core forward, dense levels)
    const PagedLevelDev* paged;   // host array of 3, or null: the levels are page pools (tensor-core forward only; L[l].n still holds the rows)
};

template <typename T> struct Elem;
template <> struct Elem<float> {
    static __device__ __forceinline__ float ld(const float* p) { return *p; }
    static __device__ __forceinline__ void st(float* p, float v) { *p = v; }
};
template <> struct Elem<__nv_bfloat16> {
    static __device__ __forceinline__ float ld(const __nv_bfloat16* p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ void st(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
};

// Rows [lo, hi) of `level` visible to key-timeline position p (L1 causal window, L2 causal prefix,
// L3 everything), clipped to [0, n).
__host__ __device__ __forceinline__ void visible_range(int level, long long p, long long W, long long n,
                                                       int decode, long long& lo, long long& hi) {
    long long a = 0, b = n;
    if (!decode) {
        if (level == 0) { a = p - W + 1; b = p + 1; }
        else if (level == 1) { b = p + 1; }
        if (a < 0) a = 0;
        if (b > n) b = n;
    }
    if (b < a) b = a;
    lo = a; hi = b;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ---- launchers implemented in the .cu files (all return a cudaError_t from the launch) ----
cudaError_t launch_router(const void* R, const float* W_r, const float* b_r, long long rows, int D, int r_dtype,
                          int route, float* gate, float* log2_gate, int8_t* idx, cudaStream_t st);
cudaError_t launch_fwd_simt(const FwdParams& p, int dtype, cudaStream_t st);

struct DecodeParams {
    const void* q;
    void* O;
    float* LSE;
    const float* gate;   // [B,3]
    LevelDev L[3];
    int B, H, d;
    int kv_group;        // query heads per KV head (>= 1)
    float scale;
    long long chunk_rows;
    long long n_chunks[3];
    long long total_chunks;
    float* partial;      // [B*H, total_chunks, d+2]
};
cudaError_t launch_decode(const DecodeParams& p, cudaStream_t st);
cudaError_t launch_decode_combine(const DecodeParams& p, cudaStream_t st);   // second kernel alone (gate, n_chunks, partial, O, LSE)

struct PagedLevelDev {
    const void* k;
    const void* v;
    const int* table;    // [B, table_stride]
    const int* rows;     // [B] or null
    long long n, table_stride, table_head_stride, sp, sh, sn;
    long long pool_pages; // pages in the pool (needed by the paged forward only)
    int page_shift;      // log2(page_rows)
};
struct DecodePagedParams {
    const void* q;
    const float* gate;   // [B,3]
    PagedLevelDev L[3];
    int B, H, H_kv, d;
    float scale;
    long long chunk_rows;
    long long n_chunks[3];
    long long total_chunks;
    float* partial;      // [B*H, total_chunks, d+2]
    unsigned int* status;              // device status word of the call's workspace (bounded waits of the copy-engine form)
    unsigned long long wait_limit_ns;
};
cudaError_t launch_decode_paged(const DecodePagedParams& p, cudaStream_t st);
cudaError_t launch_l3_index(const void* k, long long n_pages, int H_kv, int page_rows, int d, long long sp, long long sh,
                            long long sn, const float* proj, int bits, unsigned int* codes, cudaStream_t st);
cudaError_t launch_l3_retrieve(const void* q, int B, int H, int H_kv, int d, const float* proj, int bits,
                               const unsigned int* codes, const int* bank, const int* bank_len, long long bank_stride,
                               int max_bank, int R, int page_rows, int* table, int* n_sel, int* rows, cudaStream_t st);

struct BwdParams {
    const void *Q, *O, *dO;
    const float* LSE;
    const float* gate;
    LevelDev L[3];
    LevelGradDev dL[3];
    void* dQ;
    float* dG;        // [B,T,3]
    float* delta;     // ws: [B,H,T]
    float* Gpart;     // ws: [B,H,T,3]
    float* stats;     // ws: room for 6 x [B,H,Tpad] floats (tensor-core path uses 4; Tpad = T rounded up to 128)
    int B, H, T, d;
    int window, q_offset;
    float scale;
    int kv_group;     // query heads per KV head (>= 1); > 1 only on the tensor-core path
    int test_stall;   // MKA_FLAG_TEST_STALL (tensor-core path): the dK/dV kernel's loader leaves out its last query tile
};
cudaError_t launch_bwd_simt(const BwdParams& p, int dtype, cudaStream_t st);
cudaError_t launch_router_bwd(const void* R, int r_dtype, const float* dG, long long rows, int D, float* dW_r,
                              float* db_r, float* partial, int n_row_chunks, cudaStream_t st);

cudaError_t launch_fuse_kv(const LevelDev L[3], const LevelGradDev& out, const float* gate, int B, int H, long long n, int d,
                           long long dst_offset, int dtype, cudaStream_t st, const int* dst_table = nullptr,
                           long long dst_table_stride = 0, int dst_page_shift = 0, const int* dst_offsets = nullptr);
cudaError_t launch_l2_summary(const void* X, void* M2, float* state, int use_state, long long n_prev, int B, long long T, int D,
                              int dtype, int kind, float beta, unsigned int* status, cudaStream_t st);
size_t l2_summary_seg_workspace(int B, long long T, int D, int dtype);
cudaError_t launch_l2_summary_seg(const void* X, void* M2, float* state, int use_state, long long n_prev, int B, long long T,
                                  int D, int dtype, int kind, float beta, unsigned int* status, void* scratch, cudaStream_t st);
cudaError_t launch_bwd_dgate(const float* Gpart, int B, int H, long long T, float* dG, cudaStream_t st);
// Tensor-core (TMA + tcgen05) backward; same contract as the forward below.
cudaError_t launch_bwd_tc(const BwdParams& p, unsigned int* status_word, cudaStream_t st);
bool bwd_tc_eligible(const BwdParams& p, int dtype);

// Tensor-core (TMA + tcgen05) forward; returns cudaErrorNotSupported when the shape is not eligible.
cudaError_t launch_fwd_tc(const FwdParams& p, unsigned int* status_word, cudaStream_t st);
bool fwd_tc_eligible(const FwdParams& p, int dtype);

}  // namespace mka
