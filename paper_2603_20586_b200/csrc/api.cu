// C-ABI entry points of the FastMKA library: host-side validation, integer bookkeeping (decode split
// table, forward tile ranges), workspace layout, and dispatch to the kernels.  See include/mka.h.
#include <string.h>

#include <atomic>

#include "common.cuh"
#include "tc_ptx.cuh"

using namespace mka;

// Process-wide limit of the device-side waits, in microseconds.
static std::atomic<uint32_t> g_wait_limit_us{1000000u};
unsigned long long mka::wait_limit_ns() { return 1000ull * g_wait_limit_us.load(std::memory_order_relaxed); }

extern "C" uint32_t mka_set_wait_limit_us(uint32_t us) {
    if (us == 0) us = 1000000u;
    if (us < 100u) us = 100u;
    if (us > 10000000u) us = 10000000u;
    return g_wait_limit_us.exchange(us, std::memory_order_relaxed);
}

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

mka_status check_shape(const mka_shape* s, bool decode) {
    if (!s) return MKA_ERR_ARG;
    if (s->dtype != MKA_BF16 && s->dtype != MKA_F32) return MKA_ERR_ARG;
    if (s->mode != MKA_MODE_FAST && s->mode != MKA_MODE_FULL) return MKA_ERR_ARG;
    if (s->B < 0 || s->H < 0 || s->T < 0) return MKA_ERR_SHAPE;
    if (s->d != 32 && s->d != 64 && s->d != 96 && s->d != 128) return MKA_ERR_SHAPE;
    if (!decode && s->window < 1) return MKA_ERR_SHAPE;
    if (!decode && s->q_offset < 0) return MKA_ERR_SHAPE;
    if (decode && s->T != 1) return MKA_ERR_SHAPE;
    if (s->kv_heads < 0 || (s->kv_heads > 0 && s->H % s->kv_heads != 0)) return MKA_ERR_SHAPE;
    return MKA_OK;
}

mka_status check_levels(const mka_shape* s, const mka_level L[3]) {
    if (!L) return MKA_ERR_ARG;
    for (int l = 0; l < 3; ++l) {
        if (L[l].n < 0) return MKA_ERR_SHAPE;
        if (L[l].n == 0) continue;
        if (!L[l].k || !L[l].v) return MKA_ERR_ARG;
        if (L[l].stride_n < s->d || L[l].stride_b < 0 || L[l].stride_h < 0) return MKA_ERR_SHAPE;
        if (s->dtype == MKA_BF16) {
            if (!aligned16(L[l].k) || !aligned16(L[l].v)) return MKA_ERR_ALIGN;
            if (L[l].stride_n % 8 || L[l].stride_b % 8 || L[l].stride_h % 8) return MKA_ERR_ALIGN;
        }
    }
    return MKA_OK;
}

int kv_group_of(const mka_shape* s) { return s->kv_heads > 0 ? s->H / s->kv_heads : 1; }
float resolve_scale(const mka_shape* s) { return s->scale > 0.f ? s->scale : 1.0f / sqrtf((float)s->d); }

void fill_levels(LevelDev out[3], const mka_level L[3]) {
    for (int l = 0; l < 3; ++l) {
        out[l].k = L[l].k; out[l].v = L[l].v; out[l].n = L[l].n;
        out[l].sb = L[l].stride_b; out[l].sh = L[l].stride_h; out[l].sn = L[l].stride_n;
    }
}

constexpr int kRouterBwdChunks = 128;

// Per-row statistics of the tensor-core backward: three arrays of [B, H, Tpad] float2, Tpad = T rounded up to 128.
size_t bwd_stats_bytes(const mka_shape* s) {
    const size_t tpad = ((size_t)s->T + 127) / 128 * 128;
    return (size_t)3 * s->B * s->H * tpad * 2 * sizeof(float);
}

}  // namespace

extern "C" {

const char* mka_status_str(mka_status s) {
    switch (s) {
        case MKA_OK: return "ok";
        case MKA_ERR_ARG: return "invalid argument";
        case MKA_ERR_SHAPE: return "invalid shape";
        case MKA_ERR_ALIGN: return "misaligned pointer or stride";
        case MKA_ERR_WORKSPACE: return "workspace missing or too small";
        case MKA_ERR_UNSUPPORTED: return "unsupported combination";
        case MKA_ERR_CUDA: return "CUDA runtime error";
        case MKA_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

mka_status mka_decode_plan(const int64_t n_level[3], int32_t B, int32_t H, int32_t d, mka_decode_plan_t* plan) {
    if (!n_level || !plan) return MKA_ERR_ARG;
    if (B < 0 || H < 0 || d <= 0) return MKA_ERR_SHAPE;
    int64_t total_rows = 0;
    for (int l = 0; l < 3; ++l) {
        if (n_level[l] < 0) return MKA_ERR_SHAPE;
        total_rows += n_level[l];
    }
    // Aim for at least ~8 CTAs per SM over the whole grid, with chunks of 128..1024 rows (multiples of
    // 128) so that every CTA streams the same number of bytes apart from each level's last chunk.
    const int64_t target_ctas = 148 * 8;
    const int64_t bh = (int64_t)B * H > 0 ? (int64_t)B * H : 1;
    int64_t rows = (total_rows * bh + target_ctas - 1) / target_ctas;   // rows per CTA to hit the target
    rows = (rows / 128) * 128;
    if (rows < 128) rows = 128;
    if (rows > 1024) rows = 1024;
    plan->chunk_rows = rows;
    plan->total_chunks = 0;
    for (int l = 0; l < 3; ++l) {
        plan->n_chunks[l] = (n_level[l] + rows - 1) / rows;
        plan->total_chunks += plan->n_chunks[l];
    }
    return MKA_OK;
}

mka_status mka_fwd_tile_range(const mka_shape* s, const int64_t n_level[3], int32_t level, int64_t q_tile,
                              mka_tile_range* out) {
    if (!s || !n_level || !out) return MKA_ERR_ARG;
    if (level < 0 || level > 2 || q_tile < 0 || q_tile * kTileM >= (s->T > 0 ? s->T : 1)) return MKA_ERR_SHAPE;
    const long long n = n_level[level], W = s->window;
    const long long m0 = q_tile * kTileM;
    const long long m1 = (m0 + kTileM - 1 < s->T - 1 ? m0 + kTileM - 1 : s->T - 1);
    const long long p_lo = m0 + s->q_offset, p_hi = m1 + s->q_offset;
    long long lo_f, hi_f, lo_l, hi_l;
    visible_range(level, p_lo, W, n, 0, lo_f, hi_f);
    visible_range(level, p_hi, W, n, 0, lo_l, hi_l);
    const long long lo = lo_f, hi = hi_l > hi_f ? hi_l : hi_f;     // union (ranges move right with p)
    if (hi <= lo) { out->first = out->end = out->full_first = out->full_end = 0; return MKA_OK; }
    out->first = lo / kTileN;
    out->end = (hi + kTileN - 1) / kTileN;
    // intersection of all rows' ranges: [lo_l, hi_f); a key tile is "full" when it lies inside it
    const long long ilo = lo_l, ihi = hi_f;
    long long ff = (ilo + kTileN - 1) / kTileN, fe = ihi / kTileN;
    if (ff < out->first) ff = out->first;
    if (fe > out->end) fe = out->end;
    if (fe < ff) fe = ff;
    out->full_first = ff;
    out->full_end = fe;
    return MKA_OK;
}

static mka_status paged_plan(const int64_t n_level[3], int32_t B, int32_t H_kv, mka_decode_plan_t* plan);

// Grouped heads in the dense decode run the grouped-query kernel (every cached row read once per KV head).
static bool decode_uses_grouped_kernel(const mka_shape* s) {
    return s->kv_heads > 0 && s->kv_heads < s->H && s->H % s->kv_heads == 0 && s->H / s->kv_heads <= 16;
}

size_t mka_workspace_bytes(const mka_shape* s, const int64_t n_level[3], int32_t which) {
    if (!s || !n_level) return 0;
    if (which == MKA_WS_FWD) return kWsHeader;
    if (which == MKA_WS_DECODE) {
        mka_decode_plan_t plan;
        if (decode_uses_grouped_kernel(s)) {
            if (paged_plan(n_level, s->B, s->kv_heads, &plan) != MKA_OK) return 0;
        } else if (mka_decode_plan(n_level, s->B, s->H, s->d, &plan) != MKA_OK) {
            return 0;
        }
        return kWsHeader + round_up((size_t)s->B * s->H * plan.total_chunks * (s->d + 2) * sizeof(float), 256);
    }
    if (which == MKA_WS_BWD) {
        size_t rows = (size_t)s->B * s->H * s->T;
        return kWsHeader + round_up(rows * sizeof(float), 256) + round_up(rows * 3 * sizeof(float), 256) +
               round_up((size_t)kRouterBwdChunks * (s->D > 0 ? s->D : 0) * 3 * sizeof(float), 256) +
               round_up(bwd_stats_bytes(s), 256);
    }
    return 0;
}

mka_status mka_router(const void* R, const float* W_r, const float* b_r, int64_t rows, int32_t D, int32_t r_dtype,
                      int32_t route, float* gate, float* log2_gate, int8_t* route_idx, void* stream) {
    if (rows < 0 || D <= 0) return MKA_ERR_SHAPE;
    if (r_dtype != MKA_BF16 && r_dtype != MKA_F32) return MKA_ERR_ARG;
    if (route < MKA_ROUTE_SOFT || route > MKA_ROUTE_TOP2) return MKA_ERR_ARG;
    if (rows == 0) return MKA_OK;
    if (!R || !W_r || !gate) return MKA_ERR_ARG;
    cudaError_t e = launch_router(R, W_r, b_r, rows, D, r_dtype, route, gate, log2_gate, route_idx,
                                  static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? MKA_OK : MKA_ERR_CUDA;
}

mka_status mka_fwd(const mka_shape* s, const void* Q, const mka_level L[3], const float* gate, void* O, float* LSE,
                   void* ws, size_t ws_bytes, void* stream) {
    mka_status st = check_shape(s, false);
    if (st != MKA_OK) return st;
    if ((st = check_levels(s, L)) != MKA_OK) return st;
    if (s->B == 0 || s->H == 0 || s->T == 0) return MKA_OK;
    if (!Q || !gate || !O) return MKA_ERR_ARG;
    if (s->dtype == MKA_BF16 && (!aligned16(Q) || !aligned16(O))) return MKA_ERR_ALIGN;
    if (!ws || ws_bytes < kWsHeader) return MKA_ERR_WORKSPACE;
    FwdParams p;
    memset(&p, 0, sizeof(p));
    p.Q = Q; p.O = O; p.LSE = LSE; p.gate = gate;
    fill_levels(p.L, L);
    p.B = s->B; p.H = s->H; p.T = s->T; p.d = s->d;
    p.window = s->window; p.q_offset = s->q_offset; p.scale = resolve_scale(s);
    p.mode = s->mode; p.decode = 0; p.kv_group = kv_group_of(s);
    p.test_stall = (s->flags & MKA_FLAG_TEST_STALL) ? 1 : 0;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(ws, 0, 16, cs) != cudaSuccess) return MKA_ERR_CUDA;
    cudaError_t e;
    if (!(s->flags & MKA_FLAG_FORCE_SIMT) && s->mode == MKA_MODE_FAST && fwd_tc_eligible(p, s->dtype))
        e = launch_fwd_tc(p, static_cast<unsigned int*>(ws), cs);
    else
        e = launch_fwd_simt(p, s->dtype, cs);
    if (e == cudaErrorNotSupported) return MKA_ERR_UNSUPPORTED;
    return e == cudaSuccess ? MKA_OK : MKA_ERR_CUDA;
}

int32_t mka_fwd_kernel_kind(const mka_shape* s, const mka_level L[3]) {
    if (check_shape(s, false) != MKA_OK || check_levels(s, L) != MKA_OK) return -1;
    FwdParams p;
    memset(&p, 0, sizeof(p));
    fill_levels(p.L, L);
    p.B = s->B; p.H = s->H; p.T = s->T; p.d = s->d; p.mode = s->mode; p.kv_group = kv_group_of(s);
    return (!(s->flags & MKA_FLAG_FORCE_SIMT) && s->mode == MKA_MODE_FAST && fwd_tc_eligible(p, s->dtype)) ? 1 : 0;
}

mka_status mka_decode(const mka_shape* s, const void* q, const mka_level L[3], const float* gate, void* O,
                      float* LSE, void* ws, size_t ws_bytes, void* stream) {
    mka_status st = check_shape(s, true);
    if (st != MKA_OK) return st;
    if (s->dtype != MKA_BF16 || s->mode != MKA_MODE_FAST) return MKA_ERR_UNSUPPORTED;
    if (s->d != 64 && s->d != 128) return MKA_ERR_SHAPE;
    if ((st = check_levels(s, L)) != MKA_OK) return st;
    if (s->B == 0 || s->H == 0) return MKA_OK;
    if (!q || !gate || !O) return MKA_ERR_ARG;
    if (!aligned16(q) || !aligned16(O)) return MKA_ERR_ALIGN;
    int64_t n_level[3] = {L[0].n, L[1].n, L[2].n};
    size_t need = mka_workspace_bytes(s, n_level, MKA_WS_DECODE);
    if (!ws || ws_bytes < need) return MKA_ERR_WORKSPACE;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (decode_uses_grouped_kernel(s)) {
        // dense levels seen as paged ones with a single page per sequence (no table: the page is the batch index)
        mka_decode_plan_t plan;
        paged_plan(n_level, s->B, s->kv_heads, &plan);
        if ((long long)s->B * s->H * plan.total_chunks > 0x7fffffffLL) return MKA_ERR_SHAPE;
        DecodePagedParams pp;
        memset(&pp, 0, sizeof(pp));
        for (int l = 0; l < 3; ++l) {
            pp.L[l].k = L[l].k; pp.L[l].v = L[l].v; pp.L[l].table = nullptr; pp.L[l].rows = nullptr; pp.L[l].n = L[l].n;
            pp.L[l].sp = L[l].stride_b; pp.L[l].sh = L[l].stride_h; pp.L[l].sn = L[l].stride_n;
            pp.L[l].page_shift = 40;
            pp.n_chunks[l] = plan.n_chunks[l];
        }
        pp.q = q; pp.gate = gate; pp.B = s->B; pp.H = s->H; pp.H_kv = s->kv_heads; pp.d = s->d; pp.scale = resolve_scale(s);
        pp.chunk_rows = plan.chunk_rows; pp.total_chunks = plan.total_chunks;
        pp.partial = reinterpret_cast<float*>(static_cast<char*>(ws) + kWsHeader);
        pp.status = static_cast<unsigned int*>(ws); pp.wait_limit_ns = wait_limit_ns();
        DecodeParams c;
        memset(&c, 0, sizeof(c));
        c.O = O; c.LSE = LSE; c.gate = gate; c.B = s->B; c.H = s->H; c.d = s->d;
        c.total_chunks = plan.total_chunks; c.partial = pp.partial;
        for (int l = 0; l < 3; ++l) c.n_chunks[l] = plan.n_chunks[l];
        if (cudaMemsetAsync(ws, 0, 16, cs) != cudaSuccess) return MKA_ERR_CUDA;
        cudaError_t e = launch_decode_paged(pp, cs);
        if (e == cudaSuccess) e = launch_decode_combine(c, cs);
        if (e == cudaErrorNotSupported) return MKA_ERR_UNSUPPORTED;
        return e == cudaSuccess ? MKA_OK : MKA_ERR_CUDA;
    }
    mka_decode_plan_t plan;
    mka_decode_plan(n_level, s->B, s->H, s->d, &plan);
    if ((long long)s->B * s->H * plan.total_chunks > 0x7fffffffLL) return MKA_ERR_SHAPE;
    DecodeParams p;
    memset(&p, 0, sizeof(p));
    p.q = q; p.O = O; p.LSE = LSE; p.gate = gate;
    fill_levels(p.L, L);
    p.B = s->B; p.H = s->H; p.d = s->d; p.scale = resolve_scale(s); p.kv_group = kv_group_of(s);
    p.chunk_rows = plan.chunk_rows;
    for (int l = 0; l < 3; ++l) p.n_chunks[l] = plan.n_chunks[l];
    p.total_chunks = plan.total_chunks;
    p.partial = reinterpret_cast<float*>(static_cast<char*>(ws) + kWsHeader);
    if (cudaMemsetAsync(ws, 0, 16, cs) != cudaSuccess) return MKA_ERR_CUDA;
    cudaError_t e = launch_decode(p, cs);
    if (e == cudaErrorNotSupported) return MKA_ERR_UNSUPPORTED;
    return e == cudaSuccess ? MKA_OK : MKA_ERR_CUDA;
}

// Split table of the paged decode.  Its CTAs are few and long-lived (two per SM, one KV head's rows each), so what
// counts is how many rounds of resident CTAs the grid makes and what every CTA pays to start (page-table slice, first
// tiles: about as long as streaming 256 rows).  Pick the chunk length, a multiple of 128 rows, with the least
// rounds x (rows + 256).
static mka_status paged_plan(const int64_t n_level[3], int32_t B, int32_t H_kv, mka_decode_plan_t* plan) {
    if (!n_level || !plan) return MKA_ERR_ARG;
    if (B < 0 || H_kv < 0) return MKA_ERR_SHAPE;
    for (int l = 0; l < 3; ++l) if (n_level[l] < 0) return MKA_ERR_SHAPE;
    const int64_t resident = 148 * 2;
    const int64_t groups = (int64_t)B * H_kv > 0 ? (int64_t)B * H_kv : 1;
    int64_t best_rows = 128, best_cost = -1;
    for (int64_t rows = 128; rows <= 8192; rows += 128) {
        int64_t chunks = 0, longest = 0;
        for (int l = 0; l < 3; ++l) {
            chunks += (n_level[l] + rows - 1) / rows;
            const int64_t len = n_level[l] < rows ? n_level[l] : rows;
            longest = len > longest ? len : longest;
        }
        const int64_t rounds = (chunks * groups + resident - 1) / resident;
        const int64_t cost = rounds * (longest + 256);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_rows = rows; }
    }
    plan->chunk_rows = best_rows;
    plan->total_chunks = 0;
    for (int l = 0; l < 3; ++l) {
        plan->n_chunks[l] = (n_level[l] + best_rows - 1) / best_rows;
        plan->total_chunks += plan->n_chunks[l];
    }
    return MKA_OK;
}

mka_status mka_fwd_paged(const mka_shape* s, int32_t H_kv, const void* Q, const mka_paged_level L[3], const float* gate,
                         void* O, float* LSE, void* ws, size_t ws_bytes, void* stream) {
    mka_status st = check_shape(s, false);
    if (st != MKA_OK) return st;
    if (s->dtype != MKA_BF16 || s->mode != MKA_MODE_FAST || (s->flags & MKA_FLAG_FORCE_SIMT)) return MKA_ERR_UNSUPPORTED;
    if (s->d != 64 && s->d != 128) return MKA_ERR_UNSUPPORTED;
    if (!L) return MKA_ERR_ARG;
    if (H_kv <= 0 || (s->H > 0 && s->H % H_kv != 0)) return MKA_ERR_SHAPE;
    if (s->H > 65535 || s->B > 65535) return MKA_ERR_SHAPE;
    FwdParams p;
    memset(&p, 0, sizeof(p));
    PagedLevelDev P[3];
    memset(P, 0, sizeof(P));
    for (int l = 0; l < 3; ++l) {
        if (L[l].n < 0 || L[l].n > 0x7fffffffLL) return MKA_ERR_SHAPE;
        p.L[l].n = L[l].n;
        if (L[l].n == 0) continue;
        if (!L[l].k || !L[l].v || !L[l].page_table) return MKA_ERR_ARG;
        const int pr = L[l].page_rows;
        if (pr < 8 || (pr & (pr - 1)) != 0) return MKA_ERR_SHAPE;
        if (L[l].pool_pages <= 0 || L[l].pool_pages > 0x7fffffffLL || L[l].table_head_stride < 0) return MKA_ERR_SHAPE;
        const int64_t width = L[l].table_head_stride > 0 ? L[l].table_head_stride : L[l].table_stride;
        if (width * pr < L[l].n) return MKA_ERR_SHAPE;
        if (L[l].stride_n < s->d || L[l].stride_page <= 0 || L[l].stride_h < 0) return MKA_ERR_SHAPE;
        if (!aligned16(L[l].k) || !aligned16(L[l].v)) return MKA_ERR_ALIGN;
        if (L[l].stride_n % 8 || L[l].stride_page % 8 || L[l].stride_h % 8) return MKA_ERR_ALIGN;
        if (H_kv > 1 && L[l].stride_h <= 0) return MKA_ERR_SHAPE;
        int shift = 0;
        while ((1 << shift) < pr) ++shift;
        P[l].k = L[l].k; P[l].v = L[l].v; P[l].table = L[l].page_table; P[l].n = L[l].n; P[l].rows = L[l].rows;
        P[l].table_stride = L[l].table_stride; P[l].table_head_stride = L[l].table_head_stride;
        P[l].sp = L[l].stride_page; P[l].sh = L[l].stride_h; P[l].sn = L[l].stride_n;
        P[l].pool_pages = L[l].pool_pages; P[l].page_shift = shift;
    }
    if (s->B == 0 || s->H == 0 || s->T == 0) return MKA_OK;
    if (!Q || !gate || !O) return MKA_ERR_ARG;
    if (!aligned16(Q) || !aligned16(O)) return MKA_ERR_ALIGN;
    if (!ws || ws_bytes < kWsHeader) return MKA_ERR_WORKSPACE;
    p.Q = Q; p.O = O; p.LSE = LSE; p.gate = gate;
    p.B = s->B; p.H = s->H; p.T = s->T; p.d = s->d;
    p.window = s->window; p.q_offset = s->q_offset; p.scale = resolve_scale(s);
    p.mode = s->mode; p.decode = 0; p.kv_group = s->H / H_kv; p.paged = P;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(ws, 0, 16, cs) != cudaSuccess) return MKA_ERR_CUDA;
    cudaError_t e = launch_fwd_tc(p, static_cast<unsigned int*>(ws), cs);
    if (e == cudaErrorNotSupported) return MKA_ERR_UNSUPPORTED;
    return e == cudaSuccess ? MKA_OK : MKA_ERR_CUDA;
}

size_t mka_decode_paged_workspace_bytes(const mka_shape* s, int32_t H_kv, const int64_t n_level[3]) {
    if (!s || !n_level || H_kv <= 0 || s->B < 0 || s->H < 0 || s->d <= 0) return 0;
    mka_decode_plan_t plan;
    if (paged_plan(n_level, s->B, H_kv, &plan) != MKA_OK) return 0;
    return kWsHeader + round_up((size_t)s->B * s->H * plan.total_chunks * (s->d + 2) * sizeof(float), 256);
}

mka_status mka_decode_paged(const mka_shape* s, int32_t H_kv, const void* q, const mka_paged_level L[3],
                            const float* gate, void* O, float* LSE, void* ws, size_t ws_bytes, void* stream) {
    mka_status st = check_shape(s, true);
    if (st != MKA_OK) return st;
    if (s->dtype != MKA_BF16 || s->mode != MKA_MODE_FAST) return MKA_ERR_UNSUPPORTED;
    if (s->d != 64 && s->d != 128) return MKA_ERR_SHAPE;
    if (!L) return MKA_ERR_ARG;
    if (H_kv <= 0 || (s->H > 0 && (s->H % H_kv != 0 || s->H / H_kv > 16))) return MKA_ERR_SHAPE;
    int64_t n_level[3];
    DecodePagedParams p;
    memset(&p, 0, sizeof(p));
    for (int l = 0; l < 3; ++l) {
        n_level[l] = L[l].n;
        if (L[l].n < 0) return MKA_ERR_SHAPE;
        if (L[l].n == 0) continue;
        if (!L[l].k || !L[l].v || !L[l].page_table) return MKA_ERR_ARG;
        const int pr = L[l].page_rows;
        if (pr <= 0 || (pr & (pr - 1)) != 0) return MKA_ERR_SHAPE;
        {   // the table of one (sequence, head) must hold the pages of n rows
            const int64_t width = L[l].table_head_stride > 0 ? L[l].table_head_stride : L[l].table_stride;
            if (width * pr < L[l].n) return MKA_ERR_SHAPE;
        }
        if (L[l].stride_n < s->d || L[l].stride_page < 0 || L[l].stride_h < 0) return MKA_ERR_SHAPE;
        if (!aligned16(L[l].k) || !aligned16(L[l].v)) return MKA_ERR_ALIGN;
        if (L[l].stride_n % 8 || L[l].stride_page % 8 || L[l].stride_h % 8) return MKA_ERR_ALIGN;
        int shift = 0;
        while ((1 << shift) < pr) ++shift;
        p.L[l].k = L[l].k; p.L[l].v = L[l].v; p.L[l].table = L[l].page_table; p.L[l].rows = L[l].rows;
        if (L[l].table_head_stride < 0) return MKA_ERR_SHAPE;
        p.L[l].n = L[l].n; p.L[l].table_stride = L[l].table_stride; p.L[l].table_head_stride = L[l].table_head_stride;
        p.L[l].sp = L[l].stride_page; p.L[l].sh = L[l].stride_h; p.L[l].sn = L[l].stride_n;
        p.L[l].page_shift = shift;
    }
    if (s->B == 0 || s->H == 0) return MKA_OK;
    if (!q || !gate || !O) return MKA_ERR_ARG;
    if (!aligned16(q) || !aligned16(O)) return MKA_ERR_ALIGN;
    const size_t need = mka_decode_paged_workspace_bytes(s, H_kv, n_level);
    if (!ws || ws_bytes < need) return MKA_ERR_WORKSPACE;
    mka_decode_plan_t plan;
    paged_plan(n_level, s->B, H_kv, &plan);
    if ((long long)s->B * s->H * plan.total_chunks > 0x7fffffffLL) return MKA_ERR_SHAPE;
    p.q = q; p.gate = gate;
    p.B = s->B; p.H = s->H; p.H_kv = H_kv; p.d = s->d; p.scale = resolve_scale(s);
    p.chunk_rows = plan.chunk_rows;
    p.total_chunks = plan.total_chunks;
    p.partial = reinterpret_cast<float*>(static_cast<char*>(ws) + kWsHeader);
    DecodeParams c;                                    // the combine kernel of the dense decode finishes the job
    memset(&c, 0, sizeof(c));
    c.O = O; c.LSE = LSE; c.gate = gate; c.B = s->B; c.H = s->H; c.d = s->d;
    c.total_chunks = plan.total_chunks; c.partial = p.partial;
    for (int l = 0; l < 3; ++l) { p.n_chunks[l] = plan.n_chunks[l]; c.n_chunks[l] = plan.n_chunks[l]; }
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(ws, 0, 16, cs) != cudaSuccess) return MKA_ERR_CUDA;
    cudaError_t e = launch_decode_paged(p, cs);
    if (e == cudaSuccess) e = launch_decode_combine(c, cs);
    if (e == cudaErrorNotSupported) return MKA_ERR_UNSUPPORTED;
    return e == cudaSuccess ? MKA_OK : MKA_ERR_CUDA;
}

mka_status mka_l3_index(const void* k_pool, int64_t n_pages, int32_t H_kv, int32_t page_rows, int32_t d,
                        int64_t stride_page, int64_t stride_h, int64_t stride_n, const float* proj, int32_t bits,
                        uint32_t* codes, void* stream) {
    if (n_pages < 0 || H_kv < 0 || page_rows <= 0) return MKA_ERR_SHAPE;
    if (d != 64 && d != 128) return MKA_ERR_SHAPE;
    if (bits != 32 && bits != 64 && bits != 128 && bits != 256) return MKA_ERR_SHAPE;
    if (n_pages == 0 || H_kv == 0) return MKA_OK;
    if (!k_pool || !proj || !codes) return MKA_ERR_ARG;
    if (stride_n < d || stride_page < 0 || stride_h < 0) return MKA_ERR_SHAPE;
    if (!aligned16(k_pool) || stride_n % 8 || stride_page % 8 || stride_h % 8) return MKA_ERR_ALIGN;
    cudaError_t e = launch_l3_index(k_pool, n_pages, H_kv, page_rows, d, stride_page, stride_h, stride_n, proj, bits, codes,
                                    static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? MKA_OK : MKA_ERR_CUDA;
}

mka_status mka_l3_retrieve(const void* q, int32_t B, int32_t H, int32_t H_kv, int32_t d, const float* proj,
                           int32_t bits, const uint32_t* codes, const int32_t* bank, const int32_t* bank_len,
                           int64_t bank_stride, int32_t max_bank, int32_t R, int32_t page_rows, int32_t* table,
                           int32_t* n_sel, int32_t* rows, void* stream) {
    if (B < 0 || H < 0 || H_kv <= 0 || (H > 0 && H % H_kv != 0)) return MKA_ERR_SHAPE;
    if (d != 64 && d != 128) return MKA_ERR_SHAPE;
    if (bits != 32 && bits != 64 && bits != 128 && bits != 256) return MKA_ERR_SHAPE;
    if (R < 1 || R > 64 || page_rows <= 0) return MKA_ERR_SHAPE;
    if (max_bank < 0 || max_bank > 98304 || bank_stride < max_bank) return MKA_ERR_SHAPE;
    if (B == 0 || H == 0) return MKA_OK;
    if (!q || !proj || !codes || !bank || !bank_len || !table) return MKA_ERR_ARG;
    cudaError_t e = launch_l3_retrieve(q, B, H, H_kv, d, proj, bits, codes, bank, bank_len, bank_stride, max_bank, R,
                                       page_rows, table, n_sel, rows, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? MKA_OK : MKA_ERR_CUDA;
}

mka_status mka_bwd(const mka_shape* s, const void* Q, const mka_level L[3], const float* gate, const void* O,
                   const float* LSE, const void* dO, const void* R, int32_t r_dtype, void* dQ,
                   const mka_level_grad dL[3], float* dG, float* dW_r, float* db_r, void* ws, size_t ws_bytes,
                   void* stream) {
    mka_status st = check_shape(s, false);
    if (st != MKA_OK) return st;
    if (s->mode != MKA_MODE_FAST) return MKA_ERR_UNSUPPORTED;
    if ((st = check_levels(s, L)) != MKA_OK) return st;
    if (!dL) return MKA_ERR_ARG;
    for (int l = 0; l < 3; ++l) {
        if (dL[l].n != L[l].n) return MKA_ERR_SHAPE;
        if (L[l].n == 0) continue;
        if (!dL[l].dk || !dL[l].dv) return MKA_ERR_ARG;
        if (dL[l].stride_n < s->d) return MKA_ERR_SHAPE;
        if (s->dtype == MKA_BF16 && (!aligned16(dL[l].dk) || !aligned16(dL[l].dv) || dL[l].stride_n % 8 ||
                                     dL[l].stride_b % 8 || dL[l].stride_h % 8))
            return MKA_ERR_ALIGN;
    }
    if ((dW_r || db_r) && r_dtype != MKA_BF16 && r_dtype != MKA_F32) return MKA_ERR_ARG;
    if (dW_r && (!R || s->D <= 0)) return MKA_ERR_ARG;
    if (s->B == 0 || s->H == 0 || s->T == 0) return MKA_OK;
    if (!Q || !gate || !O || !LSE || !dO || !dQ || !dG) return MKA_ERR_ARG;
    if (s->dtype == MKA_BF16 && (!aligned16(Q) || !aligned16(O) || !aligned16(dO) || !aligned16(dQ))) return MKA_ERR_ALIGN;
    int64_t n_level[3] = {L[0].n, L[1].n, L[2].n};
    size_t need = mka_workspace_bytes(s, n_level, MKA_WS_BWD);
    if (!ws || ws_bytes < need) return MKA_ERR_WORKSPACE;
    const size_t rows = (size_t)s->B * s->H * s->T;
    char* w = static_cast<char*>(ws) + kWsHeader;
    BwdParams p;
    memset(&p, 0, sizeof(p));
    p.Q = Q; p.O = O; p.dO = dO; p.LSE = LSE; p.gate = gate; p.dQ = dQ; p.dG = dG;
    fill_levels(p.L, L);
    for (int l = 0; l < 3; ++l) {
        p.dL[l].dk = dL[l].dk; p.dL[l].dv = dL[l].dv; p.dL[l].n = dL[l].n;
        p.dL[l].sb = dL[l].stride_b; p.dL[l].sh = dL[l].stride_h; p.dL[l].sn = dL[l].stride_n;
    }
    p.delta = reinterpret_cast<float*>(w);
    w += round_up(rows * sizeof(float), 256);
    p.Gpart = reinterpret_cast<float*>(w);
    w += round_up(rows * 3 * sizeof(float), 256);
    float* rpart = reinterpret_cast<float*>(w);
    w += round_up((size_t)kRouterBwdChunks * (s->D > 0 ? s->D : 0) * 3 * sizeof(float), 256);
    p.stats = reinterpret_cast<float*>(w);
    p.B = s->B; p.H = s->H; p.T = s->T; p.d = s->d;
    p.window = s->window; p.q_offset = s->q_offset; p.scale = resolve_scale(s); p.kv_group = kv_group_of(s);
    p.test_stall = (s->flags & MKA_FLAG_TEST_STALL) ? 1 : 0;
    const bool tc = !(s->flags & MKA_FLAG_FORCE_SIMT) && bwd_tc_eligible(p, s->dtype);
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(ws, 0, 16, cs) != cudaSuccess) return MKA_ERR_CUDA;
    cudaError_t e;
    if (tc)
        e = launch_bwd_tc(p, static_cast<unsigned int*>(ws), cs);
    else
        e = launch_bwd_simt(p, s->dtype, cs);
    if (e == cudaErrorNotSupported) return MKA_ERR_UNSUPPORTED;
    if (e != cudaSuccess) return MKA_ERR_CUDA;
    if (dW_r || db_r) {
        e = launch_router_bwd(R, r_dtype, dG, (long long)s->B * s->T, s->D, dW_r, db_r, rpart, kRouterBwdChunks, cs);
        if (e != cudaSuccess) return MKA_ERR_CUDA;
    }
    return MKA_OK;
}

mka_status mka_fuse_kv(int32_t B, int32_t H, int64_t n, int32_t d, int32_t dtype, const mka_level L[3], const float* gate,
                       const mka_level_grad* dst, int64_t dst_offset, void* stream) {
    if (dtype != MKA_BF16 && dtype != MKA_F32) return MKA_ERR_ARG;
    if (!L || !dst) return MKA_ERR_ARG;
    if (B < 0 || H < 0 || n < 0 || dst_offset < 0) return MKA_ERR_SHAPE;
    const int elems = dtype == MKA_BF16 ? 8 : 4;
    if (d <= 0 || d > 1024 || d % elems) return MKA_ERR_SHAPE;
    if (dst->n < dst_offset + n) return MKA_ERR_SHAPE;
    if (B == 0 || H == 0 || n == 0) return MKA_OK;
    if (!gate || !dst->dk || !dst->dv) return MKA_ERR_ARG;
    if (dst->stride_n < d || dst->stride_b < 0 || dst->stride_h < 0) return MKA_ERR_SHAPE;
    if (!aligned16(dst->dk) || !aligned16(dst->dv) || dst->stride_n % elems || dst->stride_b % elems || dst->stride_h % elems)
        return MKA_ERR_ALIGN;
    int present = 0;
    LevelDev lv[3];
    for (int l = 0; l < 3; ++l) {
        if (L[l].n != 0 && L[l].n != n) return MKA_ERR_SHAPE;
        lv[l].k = L[l].k; lv[l].v = L[l].v; lv[l].n = L[l].n;
        lv[l].sb = L[l].stride_b; lv[l].sh = L[l].stride_h; lv[l].sn = L[l].stride_n;
        if (L[l].n == 0) continue;
        ++present;
        if (!L[l].k || !L[l].v) return MKA_ERR_ARG;
        if (L[l].stride_n < d || L[l].stride_b < 0 || L[l].stride_h < 0) return MKA_ERR_SHAPE;
        if (!aligned16(L[l].k) || !aligned16(L[l].v) || L[l].stride_n % elems || L[l].stride_b % elems || L[l].stride_h % elems)
            return MKA_ERR_ALIGN;
    }
    if (!present) return MKA_ERR_ARG;
    LevelGradDev out;
    out.dk = dst->dk; out.dv = dst->dv; out.n = dst->n;
    out.sb = dst->stride_b; out.sh = dst->stride_h; out.sn = dst->stride_n;
    cudaError_t e = launch_fuse_kv(lv, out, gate, B, H, n, d, dst_offset, dtype, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? MKA_OK : MKA_ERR_CUDA;
}

size_t mka_l2_summary_workspace_bytes(int32_t B, int64_t T, int32_t D, int32_t dtype) {
    if (B < 0 || T < 0 || D < 0 || (dtype != MKA_BF16 && dtype != MKA_F32)) return 0;
    return kWsHeader + l2_summary_seg_workspace(B, T, D, dtype);
}

int32_t mka_l2_summary_kernel_kind(int32_t B, int64_t T, int32_t D, int32_t dtype, size_t ws_bytes) {
    if (B <= 0 || T <= 0 || D <= 0 || (dtype != MKA_BF16 && dtype != MKA_F32)) return 0;
    const long long strips128 = (long long)B * ((D * (dtype == MKA_BF16 ? 2 : 4) + 127) / 128);
    // Measured: bf16 inputs gain from the segmented form at any width; fp32 rows are twice as many bytes, and the strip
    // form already streams them well once there are about a hundred strips.
    const bool narrow = dtype == MKA_BF16 || strips128 < 96;
    return T >= 512 && narrow && ws_bytes >= kWsHeader + l2_summary_seg_workspace(B, T, D, dtype) ? 1 : 0;
}

mka_status mka_fuse_kv_paged(int32_t B, int32_t H, int64_t n, int32_t d, int32_t dtype, const mka_level L[3],
                             const float* gate, const mka_paged_level* dst, int64_t dst_offset, const int32_t* dst_offsets,
                             void* stream) {
    if (dtype != MKA_BF16 && dtype != MKA_F32) return MKA_ERR_ARG;
    if (!L || !dst) return MKA_ERR_ARG;
    if (B < 0 || H < 0 || n < 0 || dst_offset < 0) return MKA_ERR_SHAPE;
    const int elems = dtype == MKA_BF16 ? 8 : 4;
    if (d <= 0 || d > 1024 || d % elems) return MKA_ERR_SHAPE;
    const int pr = dst->page_rows;
    if (pr <= 0 || (pr & (pr - 1)) != 0) return MKA_ERR_SHAPE;
    if (dst->table_stride * pr < dst_offset + n || dst->n < dst_offset + n) return MKA_ERR_SHAPE;   // without the per-sequence offsets
    if (B == 0 || H == 0 || n == 0) return MKA_OK;
    if (!gate || !dst->k || !dst->v || !dst->page_table) return MKA_ERR_ARG;
    if (dst->stride_n < d || dst->stride_page < 0 || dst->stride_h < 0) return MKA_ERR_SHAPE;
    if (!aligned16(dst->k) || !aligned16(dst->v) || dst->stride_n % elems || dst->stride_page % elems || dst->stride_h % elems)
        return MKA_ERR_ALIGN;
    int present = 0;
    LevelDev lv[3];
    for (int l = 0; l < 3; ++l) {
        if (L[l].n != 0 && L[l].n != n) return MKA_ERR_SHAPE;
        lv[l].k = L[l].k; lv[l].v = L[l].v; lv[l].n = L[l].n;
        lv[l].sb = L[l].stride_b; lv[l].sh = L[l].stride_h; lv[l].sn = L[l].stride_n;
        if (L[l].n == 0) continue;
        ++present;
        if (!L[l].k || !L[l].v) return MKA_ERR_ARG;
        if (L[l].stride_n < d || L[l].stride_b < 0 || L[l].stride_h < 0) return MKA_ERR_SHAPE;
        if (!aligned16(L[l].k) || !aligned16(L[l].v) || L[l].stride_n % elems || L[l].stride_b % elems || L[l].stride_h % elems)
            return MKA_ERR_ALIGN;
    }
    if (!present) return MKA_ERR_ARG;
    LevelGradDev out;
    out.dk = const_cast<void*>(dst->k); out.dv = const_cast<void*>(dst->v); out.n = dst->n;
    out.sb = dst->stride_page; out.sh = dst->stride_h; out.sn = dst->stride_n;
    int shift = 0;
    while ((1 << shift) < pr) ++shift;
    cudaError_t e = launch_fuse_kv(lv, out, gate, B, H, n, d, dst_offset, dtype, static_cast<cudaStream_t>(stream),
                                   dst->page_table, dst->table_stride, shift, dst_offsets);
    return e == cudaSuccess ? MKA_OK : MKA_ERR_CUDA;
}

mka_status mka_l2_summary(const void* X, int32_t B, int64_t T, int32_t D, int32_t dtype, int32_t kind, float beta, float* state,
                          int64_t n_prev, void* M2, void* ws, size_t ws_bytes, void* stream) {
    if (dtype != MKA_BF16 && dtype != MKA_F32) return MKA_ERR_ARG;
    const int32_t stall = kind & MKA_SUMMARY_TEST_STALL;
    kind &= ~MKA_SUMMARY_TEST_STALL;
    if (kind != MKA_SUMMARY_MEAN && kind != MKA_SUMMARY_EMA) return MKA_ERR_ARG;
    if (B < 0 || T < 0 || D < 0 || n_prev < 0 || B > 65535) return MKA_ERR_SHAPE;
    if (T > 0x7fffff00LL) return MKA_ERR_SHAPE;
    if (D % (dtype == MKA_BF16 ? 8 : 4)) return MKA_ERR_SHAPE;
    if (kind == MKA_SUMMARY_EMA && !(beta >= 0.f && beta <= 1.f)) return MKA_ERR_ARG;
    if (B == 0 || T == 0 || D == 0) return MKA_OK;
    if (!X || !M2) return MKA_ERR_ARG;
    if (n_prev > 0 && !state) return MKA_ERR_ARG;
    if (!aligned16(X) || !aligned16(M2)) return MKA_ERR_ALIGN;
    if (ws && ws_bytes < kWsHeader) return MKA_ERR_WORKSPACE;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (ws && cudaMemsetAsync(ws, 0, 16, cs) != cudaSuccess) return MKA_ERR_CUDA;
    // With enough scratch the segmented (look-back) form cuts the sequences into 256-row segments, which keeps the GPU
    // busy however few column strips there are; otherwise one CTA walks each strip from end to end.
    const bool segmented = ws && (reinterpret_cast<uintptr_t>(ws) & 15) == 0 && mka_l2_summary_kernel_kind(B, T, D, dtype, ws_bytes) == 1;
    cudaError_t e = segmented
        ? launch_l2_summary_seg(X, M2, state, n_prev > 0 ? 1 : 0, n_prev, B, T, D, dtype, kind | stall, beta,
                                static_cast<unsigned int*>(ws), static_cast<char*>(ws) + kWsHeader, cs)
        : launch_l2_summary(X, M2, state, n_prev > 0 ? 1 : 0, n_prev, B, T, D, dtype, kind, beta,
                            static_cast<unsigned int*>(ws), cs);
    if (e == cudaErrorNotSupported) return MKA_ERR_UNSUPPORTED;
    return e == cudaSuccess ? MKA_OK : MKA_ERR_CUDA;
}

int32_t mka_bwd_kernel_kind(const mka_shape* s, const mka_level L[3], const mka_level_grad dL[3]) {
    if (check_shape(s, false) != MKA_OK || check_levels(s, L) != MKA_OK || s->mode != MKA_MODE_FAST) return -1;
    BwdParams p;
    memset(&p, 0, sizeof(p));
    fill_levels(p.L, L);
    for (int l = 0; l < 3; ++l) {
        p.dL[l].sn = dL ? dL[l].stride_n : L[l].stride_n;
        p.dL[l].sh = dL ? dL[l].stride_h : L[l].stride_h;
        p.dL[l].sb = dL ? dL[l].stride_b : L[l].stride_b;
    }
    p.B = s->B; p.H = s->H; p.T = s->T; p.d = s->d; p.kv_group = kv_group_of(s);
    return (!(s->flags & MKA_FLAG_FORCE_SIMT) && bwd_tc_eligible(p, s->dtype)) ? 1 : 0;
}

mka_status mka_device_status(const void* ws, void* stream) {
    if (!ws) return MKA_ERR_ARG;
    unsigned int word = 0;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost, cs) != cudaSuccess) return MKA_ERR_CUDA;
    if (cudaStreamSynchronize(cs) != cudaSuccess) return MKA_ERR_CUDA;
    return word == 0 ? MKA_OK : MKA_ERR_TIMEOUT;
}

}  // extern "C"
