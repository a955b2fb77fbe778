// Route-fusion of Alg. 2 (step 6, and by linearity of the K/V projections steps 6-8 on projected levels):
//     out[b,h,dst_offset + j,:] = sum_l gate[b,j,l] * L_l[b,h,j,:]        for the K and for the V tensors
// with the three levels token-aligned and the gate that of the row's own token.  HBM-bound element-wise work:
// one thread owns one 16-byte vector of a row (8 bf16 or 4 fp32) of K and of V, reads it from up to three levels
// with streaming loads, accumulates in fp32 and rounds once.  Consecutive threads take consecutive vectors of a
// row, so every warp instruction moves 512 contiguous bytes.
#include "common.cuh"

namespace mka {
namespace {

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

template <typename T> struct Vec;
template <> struct Vec<__nv_bfloat16> {
    static constexpr int kElems = 8;
    static __device__ __forceinline__ void acc(const uint4& u, float w, float (&a)[8]) {
        const uint32_t x[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            a[2 * i] = fmaf(w, __uint_as_float(x[i] << 16), a[2 * i]);
            a[2 * i + 1] = fmaf(w, __uint_as_float(x[i] & 0xffff0000u), a[2 * i + 1]);
        }
    }
    static __device__ __forceinline__ uint4 pack(const float (&a)[8]) {
        uint4 r;
        uint32_t* o = reinterpret_cast<uint32_t*>(&r);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 v = __floats2bfloat162_rn(a[2 * i], a[2 * i + 1]);
            o[i] = *reinterpret_cast<const uint32_t*>(&v);
        }
        return r;
    }
};
template <> struct Vec<float> {
    static constexpr int kElems = 4;
    static __device__ __forceinline__ void acc(const uint4& u, float w, float (&a)[8]) {
        a[0] = fmaf(w, __uint_as_float(u.x), a[0]); a[1] = fmaf(w, __uint_as_float(u.y), a[1]);
        a[2] = fmaf(w, __uint_as_float(u.z), a[2]); a[3] = fmaf(w, __uint_as_float(u.w), a[3]);
    }
    static __device__ __forceinline__ uint4 pack(const float (&a)[8]) {
        return make_uint4(__float_as_uint(a[0]), __float_as_uint(a[1]), __float_as_uint(a[2]), __float_as_uint(a[3]));
    }
};

struct FuseParams {
    LevelDev L[3];        // n = rows of the level (0: absent)
    LevelGradDev out;     // dk, dv = destinations; strides in elements
    const float* gate;    // [B, n, 3]
    long long n, dst_offset;
    int B, H, d;
    // paged destination (dst_table != null): out.sb is then the stride between PAGES and row r of sequence b lives
    // in page dst_table[b * dst_table_stride + r / page_rows]
    const int* dst_table;
    const int* dst_offsets;      // per-sequence offset added to dst_offset, or null
    long long dst_table_stride;
    int dst_page_shift;
};

template <typename T>
__global__ void __launch_bounds__(256) fuse_kv_kernel(const FuseParams p, const long long total_vecs) {
    constexpr int E = Vec<T>::kElems;
    const int vpr = p.d / E;                                     // vectors per row
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total_vecs; i += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(i % vpr) * E;
        const long long row = i / vpr;                           // over B*H*n
        const long long j = row % p.n;
        const long long bh = row / p.n;
        const int h = (int)(bh % p.H), b = (int)(bh / p.H);
        const float* g = p.gate + ((long long)b * p.n + j) * 3;
        float ak[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, av[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        uint4 kk[3], vv[3];
        float w[3];
#pragma unroll
        for (int l = 0; l < 3; ++l) {                             // issue every load before the first use
            w[l] = p.L[l].n > 0 ? g[l] : 0.f;
            if (p.L[l].n > 0) {
                const long long off = b * p.L[l].sb + h * p.L[l].sh + j * p.L[l].sn + c;
                kk[l] = ld_stream16(static_cast<const T*>(p.L[l].k) + off);
                vv[l] = ld_stream16(static_cast<const T*>(p.L[l].v) + off);
            } else {
                kk[l] = vv[l] = make_uint4(0u, 0u, 0u, 0u);
            }
        }
#pragma unroll
        for (int l = 0; l < 3; ++l) {
            if (w[l] != 0.f) {                                    // a zero gate drops the level exactly (also NaN/inf in it)
                Vec<T>::acc(kk[l], w[l], ak);
                Vec<T>::acc(vv[l], w[l], av);
            }
        }
        long long oo;
        if (p.dst_table) {
            const long long r = p.dst_offset + (p.dst_offsets ? p.dst_offsets[b] : 0) + j;
            const long long page = p.dst_table[b * p.dst_table_stride + (r >> p.dst_page_shift)];
            oo = page * p.out.sb + h * p.out.sh + (r & ((1LL << p.dst_page_shift) - 1)) * p.out.sn + c;
        } else {
            oo = b * p.out.sb + h * p.out.sh + (p.dst_offset + j) * p.out.sn + c;
        }
        *reinterpret_cast<uint4*>(static_cast<T*>(p.out.dk) + oo) = Vec<T>::pack(ak);
        *reinterpret_cast<uint4*>(static_cast<T*>(p.out.dv) + oo) = Vec<T>::pack(av);
    }
}

}  // namespace

cudaError_t launch_fuse_kv(const LevelDev L[3], const LevelGradDev& out, const float* gate, int B, int H, long long n, int d,
                           long long dst_offset, int dtype, cudaStream_t st, const int* dst_table, long long dst_table_stride,
                           int dst_page_shift, const int* dst_offsets) {
    FuseParams p;
    for (int l = 0; l < 3; ++l) p.L[l] = L[l];
    p.out = out; p.gate = gate; p.n = n; p.dst_offset = dst_offset; p.B = B; p.H = H; p.d = d;
    p.dst_table = dst_table; p.dst_table_stride = dst_table_stride; p.dst_page_shift = dst_page_shift; p.dst_offsets = dst_offsets;
    const int elems = dtype == MKA_BF16 ? 8 : 4;
    const long long total = (long long)B * H * n * (d / elems);
    if (total == 0) return cudaSuccess;
    long long blocks = (total + 255) / 256;
    const long long cap = 148LL * 8 * 8;                          // a few waves of resident CTAs; the loop strides over the rest
    if (blocks > cap) blocks = cap;
    if (dtype == MKA_BF16) fuse_kv_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, st>>>(p, total);
    else fuse_kv_kernel<float><<<(unsigned)blocks, 256, 0, st>>>(p, total);
    return cudaGetLastError();
}

}  // namespace mka
