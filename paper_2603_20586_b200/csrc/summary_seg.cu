// Causal L2 session summary, segmented form: the scan of summary.cu for inputs that offer too few column strips to
// fill the GPU (one long sequence).  The sequence is cut into segments of 256 or 512 rows; a tile is one segment of one
// 128- or 64-byte column strip (32 KB, read from DRAM once into shared memory).  Persistent CTAs take tiles from a ticket
// counter and, per tile,
//   1. total their rows with a zero incoming state: the segment acts on the carried state as the affine pair
//      (a, b) = (beta^rows, total) [prefix mean: (1, sum)]; publish b and raise the segment's flag to AGGREGATE;
//   2. look back over the preceding segments of the strip, eight records at a time: the nearest segment that has
//      published its INCLUSIVE state ends the walk, the nearer ones contribute their aggregates; publish the own
//      inclusive state.  A record is one 8-byte word (flag and fp32 value together), so no fence is involved;
//   3. scan the rows again from the true incoming state and store them straight from registers.
// A CTA holds one tile at a time; six CTAs share an SM, so that some load while others scan.  Tickets are handed out in
// segment-major order and a CTA works through its tickets in order, so every segment a CTA can wait for is held by a
// running CTA; each wait is bounded all the same, and on expiry the CTA reports MKA_ERR_TIMEOUT and returns.
// Everything is fp32, and the carried states are folded in sequence order whatever the look-back met, so results are
// deterministic.
#include "tc_ptx.cuh"

namespace mka {
namespace {

constexpr int kSegThreads = 128;
constexpr int kSegCtasPerSm = 6;                     // one 32 KB tile each
constexpr int kSegTileBytes = 32768;                 // a tile: WB bytes of every row of a segment of 32768 / WB rows
constexpr int kSegMinRows = 256;                     // the shortest segment (WB = 128): sizes the scratch
constexpr int kSegBoxRows = 256;                     // rows of one TMA box; a tile is one or two of them
constexpr unsigned kFlagAggregate = 1u, kFlagInclusive = 2u;

struct SegParams {
    void* M2;
    float* state;            // [B, D] in/out, may be null
    unsigned long long* rec; // [B, S, D] one record per segment and column: flag << 32 | fp32 bits; zero before the launch
    unsigned int* ticket;    // place counter, zero before the launch
    long long T, n_prev;
    int B, D, S, strips, kind;
    float beta;
    int use_state;
    unsigned int* status;
    unsigned long long wait_limit_ns;
    int test_stall;          // test hook (MKA_SUMMARY_TEST_STALL): segment 1 of every strip never publishes its records
};

template <typename T> struct Pair2;
template <> struct Pair2<__nv_bfloat16> {
    using type = uint32_t;
    static __device__ __forceinline__ void unpack(uint32_t w, float& lo, float& hi) { lo = __uint_as_float(w << 16); hi = __uint_as_float(w & 0xffff0000u); }
    static __device__ __forceinline__ uint32_t pack(float lo, float hi) {
        const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<const uint32_t*>(&v);
    }
};
template <> struct Pair2<float> {
    using type = float2;
    static __device__ __forceinline__ void unpack(float2 w, float& lo, float& hi) { lo = w.x; hi = w.y; }
    static __device__ __forceinline__ float2 pack(float lo, float hi) { return make_float2(lo, hi); }
};

// Eight bytes of a row: four bf16 or two fp32 columns, the unit a thread loads and stores.
template <typename T> struct Oct;
template <> struct Oct<__nv_bfloat16> {
    using type = uint2;
    static constexpr int kCols = 4;
    static __device__ __forceinline__ void unpack(uint2 w, float* x) {
        x[0] = __uint_as_float(w.x << 16); x[1] = __uint_as_float(w.x & 0xffff0000u);
        x[2] = __uint_as_float(w.y << 16); x[3] = __uint_as_float(w.y & 0xffff0000u);
    }
    static __device__ __forceinline__ uint2 pack(const float* v) {
        return make_uint2(Pair2<__nv_bfloat16>::pack(v[0], v[1]), Pair2<__nv_bfloat16>::pack(v[2], v[3]));
    }
};
template <> struct Oct<float> {
    using type = float2;
    static constexpr int kCols = 2;
    static __device__ __forceinline__ void unpack(float2 w, float* x) { x[0] = w.x; x[1] = w.y; }
    static __device__ __forceinline__ float2 pack(const float* v) { return make_float2(v[0], v[1]); }
};

// A record travels as one 8-byte word, so its flag and value are always seen together and no fence is needed; a
// thread moves the records of its column pair with one 16-byte access made of two such words.
__device__ __forceinline__ void ld_rec2(const unsigned long long* p, unsigned long long& r0, unsigned long long& r1) {
    asm volatile("ld.relaxed.gpu.global.v2.b64 {%0, %1}, [%2];" : "=l"(r0), "=l"(r1) : "l"(p) : "memory");
}
__device__ __forceinline__ void st_rec2(unsigned long long* p, unsigned flag, float2 v) {
    const unsigned long long r0 = ((unsigned long long)flag << 32) | __float_as_uint(v.x);
    const unsigned long long r1 = ((unsigned long long)flag << 32) | __float_as_uint(v.y);
    asm volatile("st.relaxed.gpu.global.v2.b64 [%0], {%1, %2};" ::"l"(p), "l"(r0), "l"(r1) : "memory");
}
__device__ __forceinline__ unsigned rec_flag(unsigned long long r) { return (unsigned)(r >> 32); }
__device__ __forceinline__ float rec_val(unsigned long long r) { return __uint_as_float((unsigned)r); }

// WB = strip width in bytes (128 or 64).  The fewer strips an input offers, the narrower they are made: segments
// of one strip that are in flight at the same time wait for each other in the look-back, and with N strips about
// 888 / N of them are (measured on [1, 32768, D] inputs: 64 strips 0.76 of the copy bandwidth, 128 strips 0.82,
// 256 strips 0.94).  A narrower strip has longer segments, so a tile stays 32 KB and a thread's share 32 rows x 8 bytes.
template <typename T, bool kEma, int WB>
__global__ void __launch_bounds__(kSegThreads, kSegCtasPerSm) l2_summary_seg_kernel(const __grid_constant__ CUtensorMap map, const SegParams p) {
    using P2 = typename Pair2<T>::type;
    constexpr int kSegRows = kSegTileBytes / WB;               // rows per segment: 256 or 512
    constexpr int kNC = WB / (int)sizeof(T);                   // columns of the strip
    constexpr int kNP = kNC / 2;                               // column pairs: what one lane of the look-back warp carries
    constexpr int CW = Oct<T>::kCols;                          // columns of one thread in the scans: 8 bytes of a row
    constexpr int kNL = kNC / CW;                              // threads across a row: 16 or 8
    constexpr int G = kSegThreads / kNL;                       // row groups: 8 or 16
    constexpr int RG = kSegRows / G;                           // rows scanned by one thread: 32
    using V8 = typename Oct<T>::type;
    constexpr uint32_t kTileBytes = kSegTileBytes;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~static_cast<uintptr_t>(127));
    __shared__ float part[G][kNC];
    __shared__ float carry[kNC];
    __shared__ float a_pow[RG + 1];                            // beta^j, j = 0..RG (EMA)
    __shared__ uint64_t full;
    __shared__ WaitCtl wait_ctl;
    __shared__ unsigned place_s;
    __shared__ int pending_s;                                  // parity of the newest load's barrier phase, or -1 before any load

    const int tid = threadIdx.x;
    const int c = tid % kNL, g = tid / kNL;
    const int Tn = (int)p.T;
    const float beta = p.beta, omb = 1.f - p.beta;
    const unsigned total = (unsigned)p.S * p.B * p.strips;
    volatile WaitCtl* abortp = &wait_ctl;
    float a_rg = 1.f;                                          // beta^RG, beta^kSegRows
    if (kEma) {
#pragma unroll
        for (int k = 0; k < RG; ++k) a_rg *= beta;
    }
    float a_full = 1.f;
    if (kEma) {
#pragma unroll
        for (int k = 0; k < G; ++k) a_full *= a_rg;
    }
    // places are segment-major: place = (seg * B + b) * strips + strip
    if (kEma && tid <= RG) {
        float a = 1.f;
        for (int j = 0; j < tid; ++j) a *= beta;
        a_pow[tid] = a;
    }
    if (tid == 0) {
        wait_ctl.abort = 0;
        wait_ctl.limit_ns = p.wait_limit_ns;
        pending_s = -1;
        mbar_init(&full, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        place_s = atomicAdd(p.ticket, 1u);
    }
    __syncthreads();
    P2* tile = reinterpret_cast<P2*>(smem);                                      // [kSegRows][kNP]

    for (int it = 0;; ++it) {
        const unsigned place = place_s;
        if (place >= total) break;
        const int strip = place % p.strips;
        const int b = (place / p.strips) % p.B;
        const int seg = place / (p.strips * p.B);
        const int col0 = strip * kNC;
        const int row0 = seg * kSegRows;
        unsigned nxt = 0;
        if (tid == 0) {
            mbar_expect_tx(&full, kTileBytes);
#pragma unroll
            for (int bx = 0; bx < kSegRows / kSegBoxRows; ++bx)
                tma_load_3d(smem + (size_t)bx * kSegBoxRows * WB, &map, col0, row0 + bx * kSegBoxRows, b, &full);
            pending_s = it & 1;
            nxt = atomicAdd(p.ticket, 1u);                     // the next place; needed only at the end of this tile
        }
        bool ok = mbar_wait(&full, it & 1, abortp);

        // ---- 1. totals of this thread's rows (zero incoming state)
        const int t0 = row0 + g * RG;
        const int left = Tn - t0;
        const int nv = left >= RG ? RG : (left > 0 ? left : 0);
        const V8* trow = reinterpret_cast<const V8*>(tile) + (size_t)g * RG * kNL + c;
        float r[CW];
#pragma unroll
        for (int j = 0; j < CW; ++j) r[j] = 0.f;
        if (ok) {
#pragma unroll
            for (int k = 0; k < RG; ++k) {
                float x[CW];
                Oct<T>::unpack(trow[k * kNL], x);
                if (nv == RG || k < nv) {
#pragma unroll
                    for (int j = 0; j < CW; ++j) r[j] = kEma ? fmaf(beta, r[j], omb * x[j]) : r[j] + x[j];
                }
            }
        }
#pragma unroll
        for (int j = 0; j < CW; ++j) part[g][c * CW + j] = r[j];
        const int seg_rows = Tn - row0 >= kSegRows ? kSegRows : Tn - row0;      // valid rows of this segment (>= 1)
        auto group_a = [&](int gg) -> float {                                    // a of row group gg of this segment
            if (!kEma) return 1.f;
            const int l2 = Tn - (row0 + gg * RG);
            return a_pow[l2 >= RG ? RG : (l2 > 0 ? l2 : 0)];
        };
        ok = __syncthreads_and(ok);
        if (!ok) break;

        // ---- 2. warp 0: segment aggregate, look-back, inclusive state.  Lane = column pair (kNP <= 32).
        unsigned long long* my_rec = p.rec + ((long long)b * p.S + seg) * p.D + col0;          // this segment's records
        if (tid < 32) {
            const int lane = tid;
            const bool col_ok = lane < kNP && col0 + 2 * lane < p.D;
            float2 tot = make_float2(0.f, 0.f);
            if (lane < kNP) {
#pragma unroll
                for (int gg = 0; gg < G; ++gg) {
                    const float a = group_a(gg);
                    const float2 pt = *reinterpret_cast<const float2*>(&part[gg][2 * lane]);
                    tot.x = kEma ? fmaf(a, tot.x, pt.x) : tot.x + pt.x;
                    tot.y = kEma ? fmaf(a, tot.y, pt.y) : tot.y + pt.y;
                }
            }
            float a_seg = a_full;                                                // beta^(rows of this segment)
            if (kEma && seg_rows != kSegRows) {
                a_seg = 1.f;
                for (int gg = 0; gg < G; ++gg) a_seg *= group_a(gg);
            }
            float2 in = make_float2(0.f, 0.f);                                   // state entering the segment
            bool wok = true;
            if (seg == 0) {
                if (lane < kNP) {
                    if (p.use_state) {
                        if (col_ok) in = *reinterpret_cast<const float2*>(p.state + (long long)b * p.D + col0 + 2 * lane);
                    } else if (kEma) {
                        Pair2<T>::unpack(tile[lane], in.x, in.y);                // m_{-1} := x_0 makes m_0 = x_0
                    }
                }
            } else {
                if (col_ok && !(p.test_stall && seg == 1)) st_rec2(my_rec + 2 * lane, kFlagAggregate, tot);
                // Look back eight segments at a time (the segment at distance d = d0 + k is record k of the window)
                // until every column has met an INCLUSIVE record with nothing unpublished nearer than it.
                // Folding runs from the far end, state(d) = a * state(d + 1) + b(d), restarting at any inclusive
                // record on the way: exactly the chain the segments would have formed one after the other, so the
                // result does not depend on where the walk ended.
                const unsigned long long* back = my_rec + 2 * lane;
                const long long seg_stride = p.D;
                unsigned long long r0[8], r1[8];
                int d0 = 1, far = 0;                                             // far: distance of the window's ending record
                const unsigned long long tstart = gtimer();
                for (;;) {
                    unsigned incl_all = 0, zero_any = 0;                         // bit k: record k inclusive in all / unpublished in some column
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        r0[k] = r1[k] = 3ull << 32;                              // before segment 0: never needed
                        if (col_ok && seg - (d0 + k) >= 0) ld_rec2(back - (long long)(d0 + k) * seg_stride, r0[k], r1[k]);
                    }
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const unsigned f0 = rec_flag(r0[k]), f1 = rec_flag(r1[k]);
                        const bool inc = !col_ok || (f0 == kFlagInclusive && f1 == kFlagInclusive);
                        const bool zer = col_ok && (f0 == 0u || f1 == 0u);
                        incl_all |= (__all_sync(0xffffffffu, inc) ? 1u : 0u) << k;
                        zero_any |= (__any_sync(0xffffffffu, zer) ? 1u : 0u) << k;
                    }
                    const int kk = incl_all ? __ffs(incl_all) - 1 : 7;
                    if ((zero_any & ((2u << kk) - 1u)) != 0u) {                   // something needed is not there yet: look again
                        if (abortp->abort || gtimer() - tstart > abortp->limit_ns) { abortp->abort = 1; wok = false; break; }
                        continue;
                    }
                    if (incl_all) { far = d0 + kk; break; }
                    d0 += 8;
                }
                auto fold = [&](unsigned long long q0, unsigned long long q1) {
                    if (rec_flag(q0) == kFlagInclusive) in.x = rec_val(q0); else in.x = fmaf(a_full, in.x, rec_val(q0));
                    if (rec_flag(q1) == kFlagInclusive) in.y = rec_val(q1); else in.y = fmaf(a_full, in.y, rec_val(q1));
                };
                if (wok && d0 == 1) {                                            // the usual case: the window in registers is enough
#pragma unroll
                    for (int k = 7; k >= 0; --k)
                        if (k <= far - 1) fold(r0[k], r1[k]);
                } else if (wok) {                                                // a long walk: read again from the far end
                    for (int dd = far; dd >= 1; dd -= 8) {
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            r0[k] = r1[k] = 0ull;
                            if (col_ok && dd - k >= 1) ld_rec2(back - (long long)(dd - k) * seg_stride, r0[k], r1[k]);
                        }
#pragma unroll
                        for (int k = 0; k < 8; ++k)
                            if (dd - k >= 1) fold(r0[k], r1[k]);
                    }
                }
            }
            wok = __all_sync(0xffffffffu, wok);
            if (wok) {
                const float2 out_state = make_float2(fmaf(a_seg, in.x, tot.x), fmaf(a_seg, in.y, tot.y));
                if (col_ok) {
                    if (!(p.test_stall && seg == 1)) st_rec2(my_rec + 2 * lane, kFlagInclusive, out_state);
                    if (seg == p.S - 1 && p.state) *reinterpret_cast<float2*>(p.state + (long long)b * p.D + col0 + 2 * lane) = out_state;
                }
                if (lane < kNP) *reinterpret_cast<float2*>(&carry[2 * lane]) = in;
            } else if (lane == 0) {
                abortp->abort = 1;
            }
        }
        __syncthreads();
        if (wait_ctl.abort) break;

        // ---- 3. scan again from the true incoming state and store: sixteen lanes cover one 128-byte row
        {
            float m[CW];
#pragma unroll
            for (int j = 0; j < CW; ++j) m[j] = carry[c * CW + j];
#pragma unroll
            for (int gg = 0; gg < G; ++gg) {
                if (gg < g) {
                    const float a = group_a(gg);
#pragma unroll
                    for (int j = 0; j < CW; ++j) m[j] = kEma ? fmaf(a, m[j], part[gg][c * CW + j]) : m[j] + part[gg][c * CW + j];
                }
            }
            float cnt = (float)(p.n_prev + (long long)t0 + 1);
            V8* orow = reinterpret_cast<V8*>(static_cast<T*>(p.M2) + ((long long)b * p.T + t0) * p.D + col0) + c;
            const long long ostride = p.D / CW;                                  // row pitch in 8-byte units
            const bool col_ok = col0 + CW * c < p.D;
#pragma unroll
            for (int k = 0; k < RG; ++k) {
                float x[CW], v[CW];
                Oct<T>::unpack(trow[k * kNL], x);
                if (kEma) {
#pragma unroll
                    for (int j = 0; j < CW; ++j) { m[j] = fmaf(beta, m[j], omb * x[j]); v[j] = m[j]; }
                } else {
                    const float inv = __fdividef(1.f, cnt);
                    cnt += 1.f;
#pragma unroll
                    for (int j = 0; j < CW; ++j) { m[j] += x[j]; v[j] = m[j] * inv; }
                }
                if (col_ok && (nv == RG || k < nv)) orow[k * ostride] = Oct<T>::pack(v);
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");           // the next load into the tile follows these reads
        if (tid == 0) place_s = nxt;                                             // everyone read the old value barriers ago
        __syncthreads();
    }
    // A CTA that gave up may still have a load in flight: wait for it (bounded) before the shared memory goes away.
    __syncthreads();
    if (tid == 0 && wait_ctl.abort) {
        if (pending_s >= 0) {
            const unsigned long long tstart = gtimer();
            while (!mbar_try(&full, (uint32_t)pending_s) && gtimer() - tstart < wait_ctl.limit_ns) {}
        }
        if (p.status) atomicExch(p.status, (unsigned int)MKA_ERR_TIMEOUT);
    }
}

template <typename T, bool kEma, int WB>
cudaError_t launch_w(const void* X, SegParams p, cudaStream_t st) {
    constexpr int kNC = WB / (int)sizeof(T);
    constexpr int kRows = kSegTileBytes / WB;
    p.S = (int)((p.T + kRows - 1) / kRows);
    p.strips = (p.D + kNC - 1) / kNC;
    const long long tiles = (long long)p.S * p.B * p.strips;
    if (tiles > 0x7fffffffLL) return cudaErrorNotSupported;
    CUtensorMap map;
    if (!make_strip_map(&map, X, sizeof(T) == 2, p.D, p.T, p.B, kNC, kSegBoxRows)) return cudaErrorNotSupported;
    const size_t smem = (size_t)kSegTileBytes + 128;
    // the ticket counter and the records this launch will use start at zero
    cudaError_t e = cudaMemsetAsync(p.ticket, 0, 256 + (size_t)p.B * p.S * p.D * sizeof(unsigned long long), st);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(l2_summary_seg_kernel<T, kEma, WB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const long long resident = (long long)kSegCtasPerSm * 148;
    l2_summary_seg_kernel<T, kEma, WB><<<(unsigned)(tiles < resident ? tiles : resident), kSegThreads, smem, st>>>(map, p);
    return cudaGetLastError();
}

// Strip width: 128 bytes when all sequences together offer about 200 strips, else 64.
template <typename T, bool kEma>
cudaError_t launch_k(const void* X, const SegParams& p, cudaStream_t st) {
    const long long strips128 = (long long)p.B * ((p.D * (long long)sizeof(T) + 127) / 128);
    if (strips128 >= 192) return launch_w<T, kEma, 128>(X, p, st);
    return launch_w<T, kEma, 64>(X, p, st);          // 32-byte strips were measured too: they lose more in DRAM efficiency than they gain
}

}  // namespace

// Scratch of the segmented form: the ticket counter and one 8-byte record per segment and column.
size_t l2_summary_seg_workspace(int B, long long T, int D, int dtype) {
    (void)dtype;
    const long long S = (T + kSegMinRows - 1) / kSegMinRows;      // the widest strips have the most segments
    return 256 + (size_t)B * S * D * sizeof(unsigned long long);
}

cudaError_t launch_l2_summary_seg(const void* X, void* M2, float* state, int use_state, long long n_prev, int B, long long T,
                                  int D, int dtype, int kind, float beta, unsigned int* status, void* scratch, cudaStream_t st) {
    if (B == 0 || T == 0 || D == 0) return cudaSuccess;
    if (!tensor_map_encoder_available()) return cudaErrorNotSupported;
    SegParams p;
    p.S = 0; p.strips = 0;                                        // set per strip width at launch
    p.ticket = static_cast<unsigned int*>(scratch);
    p.rec = reinterpret_cast<unsigned long long*>(static_cast<char*>(scratch) + 256);
    p.M2 = M2; p.state = state; p.T = T; p.n_prev = n_prev; p.B = B; p.D = D; p.kind = kind; p.beta = beta;
    p.use_state = use_state; p.status = status; p.wait_limit_ns = wait_limit_ns();
    p.test_stall = (kind & MKA_SUMMARY_TEST_STALL) ? 1 : 0;
    kind &= ~MKA_SUMMARY_TEST_STALL;
    if (dtype == MKA_F32) return kind == MKA_SUMMARY_EMA ? launch_k<float, true>(X, p, st) : launch_k<float, false>(X, p, st);
    return kind == MKA_SUMMARY_EMA ? launch_k<__nv_bfloat16, true>(X, p, st) : launch_k<__nv_bfloat16, false>(X, p, st);
}

}  // namespace mka
