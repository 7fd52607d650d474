// Device code of the ReTopK decode step (sm_100a).
//
// Three kernels per step, all reading caller-owned bf16 q / K / V:
//   reuse_kernel   one CTA per (sequence, query head): normalise the query, cosine
//                  similarity to the cached queries (Eq. 6), Top-r recall and rho_max
//                  (Eq. 7), path decision (Eq. 13), insert of the normalised query.  A
//                  head on the reuse path then stays in this CTA to the end: candidate
//                  union (Eq. 8-9) in a shared-memory bitmap, exact scores of the gathered
//                  key rows (Eq. 10), Top-K (Eq. 11), softmax.V (Eq. 12), support insert.
//                  A head on the exact path only flags its KV group and leaves.
//   scan_kernel    persistent CTAs over the flagged KV groups: full-history scores
//                  e_i = q.k_i/sqrt(d) (Eq. 4); every key row streams once through the
//                  tensor cores for all G query heads of its group.
//   exact_finish_kernel  one CTA per exact-path head: global Top-K (Eq. 1) of the scanned
//                  scores by threshold collection + radix select, softmax.V (Eq. 12),
//                  support insert.  Exact Top-K attention is scan + this kernel.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

namespace retopk {

constexpr int PATH_REUSE = 0, PATH_FALLBACK = 1, PATH_REFRESH = 2;
constexpr int MODE_RETOPK = 0, MODE_EXACT = 1;

constexpr int REUSE_THREADS = 1024;
constexpr int EXACT_THREADS = 1024;
constexpr int SCAN_THREADS = 256;
constexpr int SCAN_TILE_ROWS = 256;  // key rows per scan work item
constexpr int MAX_GROUPS = 4096;     // B * H_kv limit (shared list in scan_kernel)
constexpr int SAMPLE_MAX = 8192;     // scores sampled to place the collection threshold
constexpr int SAMPLE_BINS = 2048;    // histogram over the top 11 bits of the score key

struct StepArgs {
    int B, Hq, Hkv, G, d, M, r, W, K, cap;
    long long max_seq_len;   // rows per KV head in k / v
    long long score_stride;  // elements per head in ws_scores (multiple of 4)
    int L;                   // seq_len of this step
    float tau, scale;
    int fill;                // cached entries = min(n_inserted, M)
    int slot;                // ring slot written by this step = n_inserted % M
    int refresh;             // 1 when Eq. 13's first case holds (known on the host)
    int mode;                // MODE_RETOPK or MODE_EXACT
    int NS;                  // entries in exact_finish_kernel's shared collection lists
    int step_id;             // call serial number; a KV group is flagged by storing it
    const uint16_t* q;
    const uint16_t* k;
    const uint16_t* v;
    uint16_t* out;
    float* qbar_cache;       // [B*Hq][M][d]
    int32_t* sup_cache;      // [B*Hq][M][K]
    uint8_t* ws_path;        // [B*Hq]
    float* ws_rho;           // [B*Hq]
    int32_t* ws_ncand;       // [B*Hq]
    int32_t* ws_gflag;       // [B*Hkv] == step_id when the group needs a full scan
    float* ws_scores;        // [B*Hq][score_stride]
    long long* counters;     // [B*Hq][4] reuse, fallback, refresh, cand_sum
    unsigned int* status;
    unsigned long long* slow_select;
    unsigned long long* scan_groups;
    int32_t* idx_out;        // MODE_EXACT only, may be null
};

// ------------------------------------------------------------------------------------
// small helpers
// ------------------------------------------------------------------------------------

// fp32 score -> unsigned key with the same order (-0.0 folded onto +0.0 first).
__device__ __forceinline__ uint32_t score_key(float s) {
    s += 0.0f;
    uint32_t u = __float_as_uint(s);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_score(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

__device__ __forceinline__ float dot8(const uint4& x, const float* qf) {
    float a = bf16_lo(x.x) * qf[0];
    a = fmaf(bf16_hi(x.x), qf[1], a);
    a = fmaf(bf16_lo(x.y), qf[2], a);
    a = fmaf(bf16_hi(x.y), qf[3], a);
    a = fmaf(bf16_lo(x.z), qf[4], a);
    a = fmaf(bf16_hi(x.z), qf[5], a);
    a = fmaf(bf16_lo(x.w), qf[6], a);
    a = fmaf(bf16_hi(x.w), qf[7], a);
    return a;
}

__device__ __forceinline__ void unpack8(const uint4& x, float* f) {
    f[0] = bf16_lo(x.x); f[1] = bf16_hi(x.x); f[2] = bf16_lo(x.y); f[3] = bf16_hi(x.y);
    f[4] = bf16_lo(x.z); f[5] = bf16_hi(x.z); f[6] = bf16_lo(x.w); f[7] = bf16_hi(x.w);
}

// Exclusive prefix sum of v over the block in thread order; `total` gets the block sum.
// s_ws: NT/32 ints of shared scratch.  Every thread of the block must call.
template <int NT>
__device__ __forceinline__ int block_excl_scan(int v, int* s_ws, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) s_ws[warp] = inc;
    __syncthreads();
    int wsum = (lane < NT / 32) ? s_ws[lane] : 0;
    int winc = wsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += t;
    }
    int wexcl = __shfl_sync(0xffffffffu, winc - wsum, warp);
    total = __shfl_sync(0xffffffffu, winc, NT / 32 - 1);
    __syncthreads();
    return wexcl + inc - v;
}

// ------------------------------------------------------------------------------------
// selection primitives
// ------------------------------------------------------------------------------------
struct SmemSrc {
    const uint32_t* key;
    const int32_t* idx;
    __device__ __forceinline__ uint32_t k(int i) const { return key[i]; }
    __device__ __forceinline__ int x(int i) const { return idx[i]; }
};
struct ScoreSrc {
    const float* sc;
    __device__ __forceinline__ uint32_t k(int i) const { return score_key(sc[i]); }
    __device__ __forceinline__ int x(int i) const { return i; }
};

// K-th largest key of src[0..n) (n > K >= 1) by four 8-bit radix passes.
// Returns the key value v and `need_eq` = how many elements equal to v belong to the top K.
// s_hist: 256 words, s_misc: 2 ints.
template <int NT, class Src>
__device__ void radix_select(const Src& src, int n, int K, uint32_t* s_hist, int* s_misc,
                             uint32_t& vstar, int& need_eq) {
    const int tid = threadIdx.x, lane = tid & 31;
    uint32_t prefix = 0, mask = 0;
    int kk = K;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = tid; i < 256; i += NT) s_hist[i] = 0;
        __syncthreads();
        for (int i = tid; i < n; i += NT) {
            const uint32_t key = src.k(i);
            if ((key & mask) == prefix) atomicAdd(&s_hist[(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (tid < 32) {
            // lane l owns digits 255-8l .. 248-8l (descending)
            int c = 0;
#pragma unroll
            for (int u = 0; u < 8; ++u) c += (int)s_hist[255 - 8 * lane - u];
            int inc = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int tt = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += tt;
            }
            int above = inc - c;
            if (above < kk && kk <= above + c) {
                int acc = above;
                for (int u = 0; u < 8; ++u) {
                    const int dgt = 255 - 8 * lane - u;
                    const int h = (int)s_hist[dgt];
                    if (kk <= acc + h) { s_misc[0] = dgt; s_misc[1] = kk - acc; break; }
                    acc += h;
                }
            }
        }
        __syncthreads();
        prefix |= (uint32_t)s_misc[0] << shift;
        mask |= 255u << shift;
        kk = s_misc[1];
        __syncthreads();
    }
    vstar = prefix;
    need_eq = kk;
}

// Write, in source order, every element with key > v and the first need_eq elements with
// key == v into s_sup_idx / s_sup_key.  Source order is ascending index, so the output is
// the support in ascending index order with ties resolved to the lower index.
template <int NT, class Src>
__device__ void ordered_emit(const Src& src, int n, uint32_t vstar, int need_eq, int32_t* s_sup_idx,
                             uint32_t* s_sup_key, int* s_ws) {
    const int tid = threadIdx.x;
    int gt_run = 0, eq_run = 0;
    for (int base = 0; base < n; base += NT) {
        const int i = base + tid;
        const bool valid = i < n;
        const uint32_t key = valid ? src.k(i) : 0u;
        const int fg = valid && key > vstar, fe = valid && key == vstar;
        int total;
        const int excl = block_excl_scan<NT>(fg | (fe << 16), s_ws, total);
        const int g_before = gt_run + (excl & 0xffff), e_before = eq_run + (excl >> 16);
        if (fg || (fe && e_before < need_eq)) {
            const int pos = g_before + (e_before < need_eq ? e_before : need_eq);
            s_sup_idx[pos] = src.x(i);
            s_sup_key[pos] = key;
        }
        gt_run += total & 0xffff;
        eq_run += total >> 16;
    }
}

// Top-K of the n listed entries (ascending index order in, ascending index order out).
template <int NT>
__device__ int select_listed(const uint32_t* s_key, const int32_t* s_idx, int n, int K,
                             int32_t* s_sup_idx, uint32_t* s_sup_key, uint32_t* s_hist, int* s_misc,
                             int* s_ws) {
    int ns;
    if (n <= K) {
        for (int i = threadIdx.x; i < n; i += NT) { s_sup_idx[i] = s_idx[i]; s_sup_key[i] = s_key[i]; }
        ns = n;
    } else {
        SmemSrc src{s_key, s_idx};
        uint32_t vstar;
        int need_eq;
        radix_select<NT>(src, n, K, s_hist, s_misc, vstar, need_eq);
        ordered_emit<NT>(src, n, vstar, need_eq, s_sup_idx, s_sup_key, s_ws);
        ns = K;
    }
    __syncthreads();
    return ns;
}

// ------------------------------------------------------------------------------------
// Eq. 12: out = sum_i softmax(e)_i v_i over the ns selected rows.
// s_w: ns floats; s_red: (NT/32) * D + NT floats; s_ws: 32 words.
// ------------------------------------------------------------------------------------
template <int D, int NT>
__device__ void attend(const uint16_t* vbase, int ns, const int32_t* s_sup_idx, const uint32_t* s_sup_key,
                       float* s_w, float* s_red, int* s_ws, uint16_t* out_row) {
    constexpr int LPR = D / 8;                  // lanes per bf16 row (16 bytes each)
    constexpr int RPW = 32 / LPR;               // rows per warp load
    constexpr int SLOTS = (NT / 32) * RPW;      // rows per block load
    constexpr int U = 8;                        // rows in flight per slot
    constexpr int NW = NT / 32;
    constexpr int PARTS = NT / D;               // second-stage partial sums
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LPR, myslot = warp * RPW + lane / LPR;

    uint32_t kmax = 0;
    for (int i = tid; i < ns; i += NT) kmax = max(kmax, s_sup_key[i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
    if (lane == 0) s_ws[warp] = (int)kmax;
    __syncthreads();
    kmax = 0;
    for (int w = 0; w < NW; ++w) kmax = max(kmax, (uint32_t)s_ws[w]);
    const float smax = key_score(kmax);
    __syncthreads();
    float wsum = 0.f;
    for (int i = tid; i < ns; i += NT) {
        const float w = expf(key_score(s_sup_key[i]) - smax);
        s_w[i] = w;
        wsum += w;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, o);
    float* s_wsf = reinterpret_cast<float*>(s_ws);
    if (lane == 0) s_wsf[warp] = wsum;
    __syncthreads();
    float denom = 0.f;
    for (int w = 0; w < NW; ++w) denom += s_wsf[w];

    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    for (int base = 0; base < ns; base += SLOTS * U) {
        uint4 x[U];
        float w[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = base + u * SLOTS + myslot;
            const bool ok = i < ns;
            w[u] = ok ? s_w[i] : 0.f;
            x[u] = ok ? ldg_stream(vbase + (size_t)s_sup_idx[i] * D + sub * 8) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            float f[8];
            unpack8(x[u], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = fmaf(w[u], f[e], acc[e]);
        }
    }
    // fixed-order reduction: row slots of a warp, then warps in groups, then groups
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
    if (lane < LPR) {
#pragma unroll
        for (int e = 0; e < 8; ++e) s_red[warp * D + sub * 8 + e] = acc[e];
    }
    __syncthreads();
    {
        const int j = tid % D, part = tid / D;
        constexpr int WPP = NW / PARTS;          // warps per part
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < WPP; ++w) s += s_red[(part * WPP + w) * D + j];
        s_red[NW * D + part * D + j] = s;
    }
    __syncthreads();
    if (tid < D) {
        float s = 0.f;
#pragma unroll
        for (int p = 0; p < PARTS; ++p) s += s_red[NW * D + p * D + tid];
        const float o = ns > 0 ? s / denom : 0.f;
        out_row[tid] = __bfloat16_as_ushort(__float2bfloat16_rn(o));
    }
}

// ------------------------------------------------------------------------------------
// reuse_kernel
// ------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(REUSE_THREADS, 1) reuse_kernel(const StepArgs a) {
    constexpr int NT = REUSE_THREADS;
    constexpr int NW = NT / 32;
    constexpr int LPR = D / 8, RPW = 32 / LPR, SLOTS = NW * RPW;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // layout (words): q[D] rho[M] sel[r] ws[32] misc[8] hist[256] sup_idx[K] sup_key[K] w[K]
    //                 | big: idx[cap] key[cap], aliased later by red[NW*D+NT] | bitmap
    float* s_q = reinterpret_cast<float*>(smem_raw);
    float* s_rho = s_q + D;
    int* s_sel = reinterpret_cast<int*>(s_rho + a.M);
    int* s_ws = s_sel + a.r;
    int* s_misc = s_ws + 32;
    uint32_t* s_hist = reinterpret_cast<uint32_t*>(s_misc + 8);
    int32_t* s_sup_idx = reinterpret_cast<int32_t*>(s_hist + 256);
    uint32_t* s_sup_key = reinterpret_cast<uint32_t*>(s_sup_idx + a.K);
    float* s_w = reinterpret_cast<float*>(s_sup_key + a.K);
    const int head_words = (D + a.M + a.r + 32 + 8 + 256 + 3 * a.K + 3) & ~3;
    int32_t* s_idx = reinterpret_cast<int32_t*>(smem_raw) + head_words;
    uint32_t* s_key = reinterpret_cast<uint32_t*>(s_idx + a.cap);
    float* s_red = reinterpret_cast<float*>(s_idx);
    const int big_words = (max(2 * a.cap, NW * D + NT) + 3) & ~3;
    uint32_t* s_bm = reinterpret_cast<uint32_t*>(s_idx) + big_words;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bh = blockIdx.x;
    const int b = bh / a.Hq, h = bh % a.Hq;
    const int bkv = b * a.Hkv + h / a.G;
    const int M = a.M, fill = a.fill, L = a.L, K = a.K;
    const int nwords = (L + 31) >> 5;

    // normalised query (text above Eq. 6) on warp 0 while the others clear the bitmap
    if (warp == 0) {
        const uint16_t* qrow = a.q + (size_t)bh * D;
        float x[D / 32], acc = 0.f;
#pragma unroll
        for (int u = 0; u < D / 32; ++u) {
            x[u] = __uint_as_float((uint32_t)qrow[lane + 32 * u] << 16);
            acc = fmaf(x[u], x[u], acc);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        const float nrm = sqrtf(acc);
#pragma unroll
        for (int u = 0; u < D / 32; ++u) s_q[lane + 32 * u] = nrm > 0.f ? x[u] / nrm : 0.f;
    } else if (!a.refresh) {
        uint4* bm4 = reinterpret_cast<uint4*>(s_bm);
        for (int w = tid - 32; w < (nwords + 3) >> 2; w += NT - 32) bm4[w] = make_uint4(0, 0, 0, 0);
    }
    __syncthreads();

    // Eq. 6: rho_c for every cached entry, four entries in flight per warp
    for (int c0 = warp; c0 < fill; c0 += NW * 4) {
        float4 x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int c = c0 + NW * u;
            x[u] = (c < fill && lane < D / 4)
                ? reinterpret_cast<const float4*>(a.qbar_cache + ((size_t)bh * M + c) * D)[lane]
                : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int c = c0 + NW * u;
            float acc = 0.f;
            if (lane < D / 4) {
                acc = x[u].x * s_q[4 * lane];
                acc = fmaf(x[u].y, s_q[4 * lane + 1], acc);
                acc = fmaf(x[u].z, s_q[4 * lane + 2], acc);
                acc = fmaf(x[u].w, s_q[4 * lane + 3], acc);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            if (lane == 0 && c < fill) s_rho[c] = acc;
        }
    }
    __syncthreads();

    // Eq. 7: rho_max and the min(r, fill) most similar slots (ties -> lower slot)
    const int n_sel = a.r < fill ? a.r : fill;
    if (warp == 0) {
        float rho_max = -CUDART_INF_F;
        for (int s = 0; s < n_sel; ++s) {
            float bv = -CUDART_INF_F;
            int bc = 0x7fffffff;
            for (int c = lane; c < fill; c += 32) {
                float v = s_rho[c];
                if (v != -CUDART_INF_F && (v > bv || (v == bv && c < bc))) { bv = v; bc = c; }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                int oc = __shfl_xor_sync(0xffffffffu, bc, o);
                if (ov > bv || (ov == bv && oc < bc)) { bv = ov; bc = oc; }
            }
            if (s == 0) rho_max = bv;
            if (lane == 0) {
                s_sel[s] = (bc == 0x7fffffff) ? -1 : bc;
                if (bc != 0x7fffffff) s_rho[bc] = -CUDART_INF_F;   // taken
            }
            __syncwarp();
        }
        if (lane == 0) reinterpret_cast<float*>(s_misc)[0] = rho_max;
    }
    __syncthreads();
    const float rho_max = reinterpret_cast<float*>(s_misc)[0];

    // Eq. 13
    int path;
    if (a.refresh) path = PATH_REFRESH;
    else if (rho_max < a.tau) path = PATH_FALLBACK;
    else path = PATH_REUSE;

    // insert the normalised query now: every similarity of this step has been taken
    if (tid < D) a.qbar_cache[((size_t)bh * M + a.slot) * D + tid] = s_q[tid];

    if (path != PATH_REUSE) {
        if (tid == 0) {
            a.ws_gflag[bkv] = a.step_id;       // same value from every head of the group
            a.ws_path[bh] = (uint8_t)path;
            a.ws_rho[bh] = rho_max;
            a.ws_ncand[bh] = L;
            a.counters[(size_t)bh * 4 + path] += 1;
        }
        return;
    }

    // Eq. 8-9: bitmap over key positions, then ordered extraction = sorted unique list
    {
        bool bad = false;
        const int E = n_sel * K;
        for (int e0 = tid; e0 < E; e0 += NT * 4) {
            int idx[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int e = e0 + u * NT;
                idx[u] = -1;
                if (e < E) {
                    const int s = e / K, c = s_sel[s];
                    if (c >= 0) idx[u] = a.sup_cache[((size_t)bh * M + c) * K + (e - s * K)];
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (idx[u] >= 0) {
                    if (idx[u] < L) atomicOr(&s_bm[idx[u] >> 5], 1u << (idx[u] & 31));
                    else bad = true;
                }
        }
        const int w_lo = L - a.W > 0 ? L - a.W : 0;
        for (int i = w_lo + tid; i < L; i += NT) atomicOr(&s_bm[i >> 5], 1u << (i & 31));
        if (bad) atomicOr(a.status, 1u);
    }
    __syncthreads();
    int n;
    {
        const int wpt = (nwords + NT - 1) / NT;
        const int w0 = tid * wpt;
        const int w1 = (w0 + wpt < nwords) ? w0 + wpt : nwords;
        int cnt = 0;
        for (int w = w0; w < w1; ++w) cnt += __popc(s_bm[w]);
        int pos = block_excl_scan<NT>(cnt, s_ws, n);
        for (int w = w0; w < w1; ++w) {
            uint32_t bits = s_bm[w];
            while (bits) {
                const int bit = __ffs(bits) - 1;
                s_idx[pos++] = w * 32 + bit;
                bits &= bits - 1;
            }
        }
    }
    if (tid == 0) {
        a.ws_path[bh] = (uint8_t)path;
        a.ws_rho[bh] = rho_max;
        a.ws_ncand[bh] = n;
        a.counters[(size_t)bh * 4 + PATH_REUSE] += 1;
        a.counters[(size_t)bh * 4 + 3] += n;
    }
    __syncthreads();

    // Eq. 10: exact current-query scores on the candidate rows only
    {
        const int sub = lane % LPR, myslot = warp * RPW + lane / LPR;
        const uint16_t* kbase = a.k + (size_t)bkv * a.max_seq_len * D;
        float qf[8];
        unpack8(*reinterpret_cast<const uint4*>(a.q + (size_t)bh * D + sub * 8), qf);
        constexpr int U = 8;
        for (int base = 0; base < n; base += SLOTS * U) {
            uint4 x[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int i = base + u * SLOTS + myslot;
                x[u] = i < n ? ldg_stream(kbase + (size_t)s_idx[i] * D + sub * 8) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int i = base + u * SLOTS + myslot;
                float acc = dot8(x[u], qf);
#pragma unroll
                for (int o = LPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
                if (sub == 0 && i < n) s_key[i] = score_key(acc * a.scale);
            }
        }
    }
    __syncthreads();

    // Eq. 11: Top-K of the candidates; insert the support
    const int ns = select_listed<NT>(s_key, s_idx, n, K, s_sup_idx, s_sup_key, s_hist, s_misc, s_ws);
    int32_t* sup_out = a.sup_cache + ((size_t)bh * M + a.slot) * K;
    for (int i = tid; i < K; i += NT) sup_out[i] = i < ns ? s_sup_idx[i] : -1;

    // Eq. 12 (s_red aliases the candidate lists, which are dead now)
    attend<D, NT>(a.v + (size_t)bkv * a.max_seq_len * D, ns, s_sup_idx, s_sup_key, s_w, s_red, s_ws,
                  a.out + (size_t)bh * D);
}

// ------------------------------------------------------------------------------------
// scan_kernel: full-history scores on the tensor cores (mma.sync m16n8k16, bf16 -> fp32)
//
// A 16-row key tile is the A operand, the group's query heads (zero padded to 8) the B
// operand.  A dot product does not care in which order its terms are paired, so each
// thread loads 16 contiguous bytes of a key row straight into its A-fragment registers
// and the query fragment is permuted to match: no shared memory, no transposes.
// CTAs are persistent: the flagged groups' rows are cut into 256-row work items and every
// CTA takes one contiguous share of them.
// ------------------------------------------------------------------------------------
__device__ __forceinline__ void mma_bf16_16816(float* c, uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int D, int NTILE>   // NTILE = ceil(G / 8) head tiles
__global__ void __launch_bounds__(SCAN_THREADS) scan_kernel(const StepArgs a) {
    constexpr int NJ = D / 32;   // 64-byte column groups per row
    __shared__ int s_list[MAX_GROUPS];
    __shared__ int s_ws[SCAN_THREADS / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int G = a.G, L = a.L;
    const int n_groups = a.B * a.Hkv;

    // the groups to scan, in ascending order (all of them for Exact Top-K attention)
    int n_act = 0;
    if (a.mode == MODE_EXACT) n_act = n_groups;
    else
        for (int base = 0; base < n_groups; base += SCAN_THREADS) {
            const int i = base + tid;
            const int f = (i < n_groups) && a.ws_gflag[i] == a.step_id;
            int total;
            const int pos = n_act + block_excl_scan<SCAN_THREADS>(f, s_ws, total);
            if (f) s_list[pos] = i;
            n_act += total;
        }
    if (n_act == 0) return;
    __syncthreads();
    if (blockIdx.x == 0 && tid == 0) atomicAdd(a.scan_groups, (unsigned long long)n_act);

    const int tpg = (L + SCAN_TILE_ROWS - 1) / SCAN_TILE_ROWS;     // work items per group
    const long long total_items = (long long)n_act * tpg;
    const long long per = (total_items + gridDim.x - 1) / gridDim.x;
    const long long it0 = (long long)blockIdx.x * per;
    const long long it1 = it0 + per < total_items ? it0 + per : total_items;

    uint32_t bq[NTILE][NJ][2][2];
    unsigned need = 0;
    int cur = -1, head0 = 0;
    const uint16_t* kbase = nullptr;
    const float scale = a.scale;

    for (long long item = it0; item < it1; ++item) {
        const int gi = (int)(item / tpg), rb = (int)(item - (long long)gi * tpg);
        const int bkv = (a.mode == MODE_EXACT) ? gi : s_list[gi];
        if (bkv != cur) {
            cur = bkv;
            const int b = bkv / a.Hkv, kvh = bkv % a.Hkv;
            head0 = b * a.Hq + kvh * G;
            kbase = a.k + (size_t)bkv * a.max_seq_len * D;
            need = 0;
            if (a.mode == MODE_EXACT) need = (1u << G) - 1u;
            else
                for (int j = 0; j < G; ++j)
                    if (a.ws_path[head0 + j] != PATH_REUSE) need |= 1u << j;
            // query fragments (B operand), permuted like the key loads below
#pragma unroll
            for (int nt = 0; nt < NTILE; ++nt) {
                const int head = nt * 8 + g;
                const uint32_t* qrow = reinterpret_cast<const uint32_t*>(a.q + (size_t)(head0 + head) * D);
#pragma unroll
                for (int j = 0; j < NJ; ++j)
#pragma unroll
                    for (int p = 0; p < 2; ++p) {
                        const int w = j * 16 + t * 4 + 2 * p;
                        bq[nt][j][p][0] = head < G ? qrow[w] : 0u;
                        bq[nt][j][p][1] = head < G ? qrow[w + 1] : 0u;
                    }
            }
        }
        // this warp's two 16-row tiles of the 256-row item; all loads first
        const int rbase = rb * SCAN_TILE_ROWS + warp * 16;
        uint4 x[2][NJ], y[2][NJ];
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            const int r0 = rbase + s * 128 + g, r1 = r0 + 8;
            const int c0 = r0 < L ? r0 : L - 1, c1 = r1 < L ? r1 : L - 1;   // never read past L
            const uint16_t* p0 = kbase + (size_t)c0 * D + t * 8;
            const uint16_t* p1 = kbase + (size_t)c1 * D + t * 8;
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
                x[s][j] = ldg_stream(p0 + j * 32);
                y[s][j] = ldg_stream(p1 + j * 32);
            }
        }
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            const int r0 = rbase + s * 128 + g, r1 = r0 + 8;
#pragma unroll
            for (int nt = 0; nt < NTILE; ++nt) {
                float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int j = 0; j < NJ; ++j) {
                    mma_bf16_16816(c, x[s][j].x, y[s][j].x, x[s][j].y, y[s][j].y, bq[nt][j][0][0], bq[nt][j][0][1]);
                    mma_bf16_16816(c, x[s][j].z, y[s][j].z, x[s][j].w, y[s][j].w, bq[nt][j][1][0], bq[nt][j][1][1]);
                }
                // c0,c1: row r0, heads 2t, 2t+1 of this tile; c2,c3: row r1
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int head = nt * 8 + 2 * t + e;
                    if (head < G && ((need >> head) & 1u)) {
                        float* srow = a.ws_scores + (size_t)(head0 + head) * a.score_stride;
                        if (r0 < L) srow[r0] = c[e] * scale;
                        if (r1 < L) srow[r1] = c[2 + e] * scale;
                    }
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------
// exact_finish_kernel
// ------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(EXACT_THREADS, 1) exact_finish_kernel(const StepArgs a) {
    constexpr int NT = EXACT_THREADS;
    constexpr int NW = NT / 32;
    const int bh = blockIdx.x;
    if (a.mode == MODE_RETOPK && a.ws_path[bh] == PATH_REUSE) return;

    extern __shared__ __align__(16) unsigned char smem_raw[];
    // layout (words): key[NS] idx[NS] (aliased later by red[NW*D+NT]) sup_idx[K] sup_key[K] w[K]
    //                 hist[SAMPLE_BINS] ws[32] misc[8] wcnt[NW] woff[NW]
    uint32_t* s_key = reinterpret_cast<uint32_t*>(smem_raw);
    int32_t* s_idx = reinterpret_cast<int32_t*>(s_key + a.NS);
    float* s_red = reinterpret_cast<float*>(smem_raw);
    int32_t* s_sup_idx = s_idx + a.NS;
    uint32_t* s_sup_key = reinterpret_cast<uint32_t*>(s_sup_idx + a.K);
    float* s_w = reinterpret_cast<float*>(s_sup_key + a.K);
    uint32_t* s_hist = reinterpret_cast<uint32_t*>(s_w + a.K);
    int* s_ws = reinterpret_cast<int*>(s_hist + SAMPLE_BINS);
    int* s_misc = s_ws + 32;
    int* s_wcnt = s_misc + 8;
    int* s_woff = s_wcnt + NW;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = bh / a.Hq, h = bh % a.Hq;
    const int bkv = b * a.Hkv + h / a.G;
    const int K = a.K, L = a.L, NS = a.NS;
    const float* sc = a.ws_scores + (size_t)bh * a.score_stride;

    int ns = -1;      // selected entries in s_sup_*; -1 = not selected yet
    int n = 0;        // collected entries in s_key / s_idx
    bool slow = false;

    if (L <= K) {
        for (int i = tid; i < L; i += NT) { s_sup_idx[i] = i; s_sup_key[i] = score_key(sc[i]); }
        ns = L;
        __syncthreads();
    } else {
        // 1. threshold from a block-strided sample, so that about 2K scores pass it
        const bool all = L <= SAMPLE_MAX;
        const int n_s = all ? L : SAMPLE_MAX;
        for (int i = tid; i < SAMPLE_BINS; i += NT) s_hist[i] = 0;
        {
            const int blk = L >> 3;
            float sv[SAMPLE_MAX / NT];
#pragma unroll
            for (int u = 0; u < SAMPLE_MAX / NT; ++u) {
                const int i = tid + u * NT;
                const int pos = all ? i : (i >> 10) * blk + (i & 1023);
                sv[u] = i < n_s ? sc[pos] : 0.f;
            }
            __syncthreads();
#pragma unroll
            for (int u = 0; u < SAMPLE_MAX / NT; ++u)
                if (tid + u * NT < n_s) atomicAdd(&s_hist[score_key(sv[u]) >> 21], 1u);
        }
        __syncthreads();
        int j;
        if (all) j = K;
        else {
            const float kf = (float)K * (float)n_s / (float)L;
            j = (int)ceilf(kf + 4.f * sqrtf(kf) + 8.f);
        }
        uint32_t thr_key = 0;
        if (j < n_s) {
            // lowest bin edge with at least j sampled scores at or above it
            constexpr int BPT = SAMPLE_BINS / NT;
            int c = 0;
#pragma unroll
            for (int u = 0; u < BPT; ++u) c += (int)s_hist[SAMPLE_BINS - 1 - BPT * tid - u];
            int total;
            const int above = block_excl_scan<NT>(c, s_ws, total);
            if (above < j && j <= above + c) {
                int acc = above;
                for (int u = 0; u < BPT; ++u) {
                    const int bin = SAMPLE_BINS - 1 - BPT * tid - u;
                    acc += (int)s_hist[bin];
                    if (acc >= j) { s_misc[2] = bin; break; }
                }
            }
            __syncthreads();
            thr_key = (uint32_t)s_misc[2] << 21;
        }

        // 2. every warp collects, in index order, the scores of its own contiguous segment
        //    that reach the threshold, into its own slice of the shared lists
        const int cap_w = NS / NW;
        const int wseg = ((L + NW * 128 - 1) / (NW * 128)) * 128;
        const int begin = warp * wseg;
        const int end = begin + wseg < L ? begin + wseg : L;
        uint32_t* wkey = s_key + warp * cap_w;
        int32_t* widx = s_idx + warp * cap_w;
        const unsigned lt = (1u << lane) - 1u;
        int cnt_w = 0;
        for (int base = begin; base < end; base += 128 * 4) {
            float4 x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i0 = base + u * 128 + lane * 4;
                x[u] = i0 < end ? *reinterpret_cast<const float4*>(sc + i0) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i0 = base + u * 128 + lane * 4;
                uint32_t key[4] = {score_key(x[u].x), score_key(x[u].y), score_key(x[u].z), score_key(x[u].w)};
                int f[4];
                unsigned bal[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    f[e] = (i0 + e < end) && key[e] >= thr_key;
                    bal[e] = __ballot_sync(0xffffffffu, f[e]);
                }
                if (bal[0] | bal[1] | bal[2] | bal[3]) {
                    int pos = cnt_w + __popc(bal[0] & lt) + __popc(bal[1] & lt) + __popc(bal[2] & lt) +
                              __popc(bal[3] & lt);
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (f[e]) {
                            if (pos < cap_w) { wkey[pos] = key[e]; widx[pos] = i0 + e; }
                            ++pos;
                        }
                    cnt_w += __popc(bal[0]) + __popc(bal[1]) + __popc(bal[2]) + __popc(bal[3]);
                }
            }
        }
        if (lane == 0) s_wcnt[warp] = cnt_w;
        __syncthreads();
        if (warp == 0) {
            const int c = s_wcnt[lane];
            int inc = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int tt = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += tt;
            }
            s_woff[lane] = inc - c;
            const unsigned over = __ballot_sync(0xffffffffu, c > cap_w);
            if (lane == 31) { s_misc[3] = inc; s_misc[4] = over != 0; }
        }
        __syncthreads();
        n = s_misc[3];
        if (s_misc[4] || n < K) slow = true;
        else {
            // 3. close the gaps between the warp slices (through registers: slices overlap targets)
            uint32_t mk[8];
            int32_t mi[8];
            const int per_thread = (NS + NT - 1) / NT;     // <= 8 for NS <= 8192; more handled below
            for (int chunk = 0; chunk < per_thread; chunk += 8) {
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int e = (chunk + u) * NT + tid;
                    const int w = e / cap_w, jj = e - w * cap_w;
                    const bool ok = e < NS && jj < s_wcnt[w];
                    mk[u] = ok ? s_key[e] : 0u;
                    mi[u] = ok ? s_idx[e] : -1;
                }
                __syncthreads();
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int e = (chunk + u) * NT + tid;
                    const int w = e / cap_w, jj = e - w * cap_w;
                    if (mi[u] >= 0) { s_key[s_woff[w] + jj] = mk[u]; s_idx[s_woff[w] + jj] = mi[u]; }
                }
                __syncthreads();
            }
        }
    }
    if (slow) {
        // multi-pass select straight from the score array (heavy ties, odd distributions)
        ScoreSrc src{sc};
        uint32_t vstar;
        int need_eq;
        radix_select<NT>(src, L, K, s_hist, s_misc, vstar, need_eq);
        ordered_emit<NT>(src, L, vstar, need_eq, s_sup_idx, s_sup_key, s_ws);
        ns = K;
        if (tid == 0) atomicAdd(a.slow_select, 1ull);
        __syncthreads();
    }
    if (ns < 0) ns = select_listed<NT>(s_key, s_idx, n, K, s_sup_idx, s_sup_key, s_hist, s_misc, s_ws);

    // record the support (cache insert / caller's index output)
    int32_t* sup_out = nullptr;
    if (a.mode == MODE_RETOPK) sup_out = a.sup_cache + ((size_t)bh * a.M + a.slot) * K;
    else if (a.idx_out) sup_out = a.idx_out + (size_t)bh * K;
    if (sup_out)
        for (int i = tid; i < K; i += NT) sup_out[i] = i < ns ? s_sup_idx[i] : -1;

    attend<D, NT>(a.v + (size_t)bkv * a.max_seq_len * D, ns, s_sup_idx, s_sup_key, s_w, s_red, s_ws,
                  a.out + (size_t)bh * D);
}

// Clear the caches (supports to -1, queries and counters to 0).
__global__ void reset_kernel(float* qbar, size_t n_q, int32_t* sup, size_t n_sup, long long* counters,
                             size_t n_cnt, int32_t* gflag, size_t n_flag, unsigned int* status,
                             unsigned long long* slow, unsigned long long* groups) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t t0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (size_t i = t0; i < n_q; i += stride) qbar[i] = 0.f;
    for (size_t i = t0; i < n_sup; i += stride) sup[i] = -1;
    for (size_t i = t0; i < n_cnt; i += stride) counters[i] = 0;
    for (size_t i = t0; i < n_flag; i += stride) gflag[i] = -1;
    if (t0 == 0) { *status = 0u; *slow = 0ull; *groups = 0ull; }
}

}  // namespace retopk
