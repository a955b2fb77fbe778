// L3 recall (Alg. 2 step 4, "L3 <- Retrieve(Q_h)"; the method section's vectorized hashing with chunk-based recall).
// The paper names the mechanism but not the hash.  Here a chunk is one page of the long-term key pool and its
// signature is a sign-random-projection code of the SUM of its keys; a query's code comes from the sum of the query
// heads that share the KV head; the R chunks whose codes agree with the query's in the most bits are recalled (ties
// to the earlier chunk) and listed in bank order as a page table for the paged decode.
// Code bits are decided by fp32 arithmetic, so its order is fixed: sums run row by row, a projection is one fmaf
// chain over the columns.
//   l3_index_kernel     HBM-bound: reads every key of the pool once, writes bits/8 bytes per (page, KV head)
//   l3_retrieve_kernel  one CTA per (sequence, KV head): query code, Hamming scores of the bank, R selection rounds
#include "common.cuh"

namespace mka {
namespace {

constexpr int kIdxThreads = 256;
constexpr int kIdxLanes = 16;                         // threads per (page, head): 8 columns each for d = 128
constexpr int kIdxPairs = kIdxThreads / kIdxLanes;    // (page, head) pairs per batch of a CTA

struct L3IndexParams {
    const __nv_bfloat16* k;
    const float* proj;       // [bits, d]
    unsigned int* codes;     // [pages, H_kv, bits / 32]
    long long n_pages, sp, sh, sn;
    int H_kv, page_rows, d, bits;
};

// dynamic shared memory: projT [d][bits] floats, then s [kIdxPairs][d] floats
__global__ void __launch_bounds__(kIdxThreads) l3_index_kernel(const L3IndexParams p) {
    extern __shared__ __align__(16) float sm[];
    float* projT = sm;
    float* s = sm + (size_t)p.d * p.bits;
    const int tid = threadIdx.x;
    for (int e = tid; e < p.d * p.bits; e += kIdxThreads) {
        const int j = e / p.d, i = e % p.d;
        projT[i * p.bits + j] = p.proj[e];
    }
    const int lane16 = tid % kIdxLanes, slot = tid / kIdxLanes;
    const int vecs = p.d / 8;                                  // 16-byte pieces of a row: 16 (d = 128) or 8 (d = 64)
    const long long pairs = p.n_pages * p.H_kv;
    const int words = p.bits / 32;
    for (long long base = (long long)blockIdx.x * kIdxPairs; base < pairs; base += (long long)gridDim.x * kIdxPairs) {
        __syncthreads();                                       // projT is there; the previous batch is done with s
        const long long pair = base + slot;
        // ---- sums of the page's keys, row by row, eight columns per thread
        if (pair < pairs && lane16 < vecs) {
            const long long pg = pair / p.H_kv, h = pair % p.H_kv;
            const __nv_bfloat16* src = p.k + pg * p.sp + h * p.sh + lane16 * 8;
            float acc[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = 0.f;
            for (int r0 = 0; r0 < p.page_rows; r0 += 8) {
                uint4 u[8];
#pragma unroll
                for (int r = 0; r < 8; ++r)
                    if (r0 + r < p.page_rows) u[r] = *reinterpret_cast<const uint4*>(src + (long long)(r0 + r) * p.sn);
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    if (r0 + r < p.page_rows) {
                        const uint32_t w[4] = {u[r].x, u[r].y, u[r].z, u[r].w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            acc[2 * i] = acc[2 * i] + __uint_as_float(w[i] << 16);
                            acc[2 * i + 1] = acc[2 * i + 1] + __uint_as_float(w[i] & 0xffff0000u);
                        }
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) s[slot * p.d + lane16 * 8 + i] = acc[i];
        }
        __syncthreads();
        // ---- projections: thread = (pair, four consecutive bits of a 64-bit group); one fmaf chain per bit
        {
            const bool valid = pair < pairs;                   // every lane runs the shuffles below
            const float* sv = s + slot * p.d;
            for (int g0 = 0; g0 < p.bits; g0 += 64) {
                const int j0 = g0 + 4 * lane16;
                float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
                if (valid && j0 < p.bits) {
                    for (int i = 0; i < p.d; ++i) {
                        const float4 pr = *reinterpret_cast<const float4*>(projT + i * p.bits + j0);
                        const float x = sv[i];
                        a0 = fmaf(pr.x, x, a0); a1 = fmaf(pr.y, x, a1); a2 = fmaf(pr.z, x, a2); a3 = fmaf(pr.w, x, a3);
                    }
                }
                unsigned nib = (a0 >= 0.f ? 1u : 0u) | (a1 >= 0.f ? 2u : 0u) | (a2 >= 0.f ? 4u : 0u) | (a3 >= 0.f ? 8u : 0u);
                if (j0 >= p.bits) nib = 0u;
                unsigned word = nib << (4 * (lane16 & 7));     // lanes 0-7 fill the group's first word, 8-15 the second
                word |= __shfl_xor_sync(0xffffffffu, word, 1);
                word |= __shfl_xor_sync(0xffffffffu, word, 2);
                word |= __shfl_xor_sync(0xffffffffu, word, 4);
                const int w = g0 / 32 + (lane16 >> 3);
                if (valid && (lane16 & 7) == 0 && w < words) p.codes[pair * words + w] = word;
            }
        }
    }
}

struct L3RetrieveParams {
    const __nv_bfloat16* q;       // [B, H, d]
    const float* proj;            // [bits, d]
    const unsigned int* codes;    // [pages, H_kv, words]
    const int* bank;              // [B, bank_stride]
    const int* bank_len;          // [B]
    int* table;                   // [B, H_kv, R]
    int* n_sel;                   // [B] or null
    int* rows;                    // [B] or null: n_sel * page_rows
    long long bank_stride;
    int B, H, H_kv, d, bits, R, page_rows, max_bank;
};

constexpr int kRetThreads = 256;
constexpr int kMaxR = 64;
constexpr unsigned short kTaken = 0xffffu;

// dynamic shared memory: unsigned short score[max_bank]
__global__ void __launch_bounds__(kRetThreads) l3_retrieve_kernel(const L3RetrieveParams p) {
    extern __shared__ __align__(16) unsigned short score[];
    __shared__ float qs[256];
    __shared__ unsigned int qcode[8];
    __shared__ unsigned long long red[kRetThreads / 32];
    __shared__ int sel[kMaxR];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x / p.H_kv, kvh = blockIdx.x % p.H_kv;
    const int G = p.H / p.H_kv, words = p.bits / 32;
    // query of the KV head: the group's heads summed in head order, fp32
    if (tid < p.d) {
        const __nv_bfloat16* q0 = p.q + ((long long)b * p.H + (long long)kvh * G) * p.d + tid;
        float acc = 0.f;
        for (int g = 0; g < G; ++g) acc = acc + __bfloat162float(q0[(long long)g * p.d]);
        qs[tid] = acc;
    }
    if (tid < 8) qcode[tid] = 0u;
    __syncthreads();
    if (tid < p.bits) {
        const float* pr = p.proj + (long long)tid * p.d;
        float acc = 0.f;
        for (int i = 0; i < p.d; ++i) acc = fmaf(pr[i], qs[i], acc);
        if (acc >= 0.f) atomicOr(&qcode[tid >> 5], 1u << (tid & 31));
    }
    __syncthreads();
    int n = p.bank_len[b];
    n = n < 0 ? 0 : (n > p.max_bank ? p.max_bank : n);
    const int* bank = p.bank + (long long)b * p.bank_stride;
    for (int c = tid; c < n; c += kRetThreads) {
        const unsigned int* code = p.codes + ((long long)bank[c] * p.H_kv + kvh) * words;
        int dist = 0;
        for (int w = 0; w < words; ++w) dist += __popc(code[w] ^ qcode[w]);
        score[c] = (unsigned short)(p.bits - dist);            // agreement: 0..bits (<= 256)
    }
    __syncthreads();
    const int k = p.R < n ? p.R : n;
    for (int r = 0; r < k; ++r) {
        // key = agreement in the high half, inverted position in the low half: the maximum is the best score, earliest chunk
        unsigned long long best = 0ull;
        for (int c = tid; c < n; c += kRetThreads) {
            const unsigned short sc = score[c];
            if (sc == kTaken) continue;
            const unsigned long long key = ((unsigned long long)(sc + 1u) << 32) | (unsigned)(0x7fffffff - c);
            best = key > best ? key : best;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
            best = other > best ? other : best;
        }
        if (lane == 0) red[warp] = best;
        __syncthreads();
        if (tid == 0) {
            unsigned long long m = red[0];
            for (int w = 1; w < kRetThreads / 32; ++w) m = red[w] > m ? red[w] : m;
            const int c = 0x7fffffff - (int)(m & 0xffffffffu);
            sel[r] = c;
            score[c] = kTaken;
        }
        __syncthreads();
    }
    if (tid == 0) {
        for (int i = 1; i < k; ++i) {                           // bank (time) order
            const int v = sel[i];
            int j = i - 1;
            while (j >= 0 && sel[j] > v) { sel[j + 1] = sel[j]; --j; }
            sel[j + 1] = v;
        }
        int* out = p.table + ((long long)b * p.H_kv + kvh) * p.R;
        for (int i = 0; i < p.R; ++i) out[i] = i < k ? bank[sel[i]] : 0;
        if (kvh == 0) {
            if (p.n_sel) p.n_sel[b] = k;
            if (p.rows) p.rows[b] = k * p.page_rows;
        }
    }
}

}  // namespace

cudaError_t launch_l3_index(const void* k, long long n_pages, int H_kv, int page_rows, int d, long long sp, long long sh,
                            long long sn, const float* proj, int bits, unsigned int* codes, cudaStream_t st) {
    if (n_pages == 0 || H_kv == 0) return cudaSuccess;
    L3IndexParams p;
    p.k = static_cast<const __nv_bfloat16*>(k); p.proj = proj; p.codes = codes;
    p.n_pages = n_pages; p.sp = sp; p.sh = sh; p.sn = sn; p.H_kv = H_kv; p.page_rows = page_rows; p.d = d; p.bits = bits;
    const size_t smem = ((size_t)d * bits + (size_t)kIdxPairs * d) * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(l3_index_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const long long batches = (n_pages * H_kv + kIdxPairs - 1) / kIdxPairs;
    const long long resident = 148LL * (smem > 100 * 1024 ? 1 : (smem > 48 * 1024 ? 2 : 4));
    // a few batches per CTA amortise the transposed projection in shared memory
    long long grid = batches < resident * 4 ? (batches + 3) / 4 : resident;
    if (grid < 1) grid = 1;
    l3_index_kernel<<<(unsigned)grid, kIdxThreads, smem, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_l3_retrieve(const void* q, int B, int H, int H_kv, int d, const float* proj, int bits,
                               const unsigned int* codes, const int* bank, const int* bank_len, long long bank_stride,
                               int max_bank, int R, int page_rows, int* table, int* n_sel, int* rows, cudaStream_t st) {
    if (B == 0 || H_kv == 0) return cudaSuccess;
    L3RetrieveParams p;
    p.q = static_cast<const __nv_bfloat16*>(q); p.proj = proj; p.codes = codes; p.bank = bank; p.bank_len = bank_len;
    p.table = table; p.n_sel = n_sel; p.rows = rows; p.bank_stride = bank_stride;
    p.B = B; p.H = H; p.H_kv = H_kv; p.d = d; p.bits = bits; p.R = R; p.page_rows = page_rows; p.max_bank = max_bank;
    const size_t smem = ((size_t)(max_bank > 0 ? max_bank : 1) * sizeof(unsigned short) + 15) / 16 * 16;
    cudaError_t e = cudaFuncSetAttribute(l3_retrieve_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    l3_retrieve_kernel<<<(unsigned)(B * H_kv), kRetThreads, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace mka
