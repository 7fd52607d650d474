// Device code of the ReTopK decode step (sm_100a).
//
// Three kernels per step, all reading caller-owned bf16 q / K / V:
//   recall_kernel  one CTA per (sequence, query head): normalise the query, cosine
//                  similarity to the cached queries (Eq. 6), Top-r recall and rho_max
//                  (Eq. 7), path decision (Eq. 13), insert of the normalised query, and
//                  on the reuse path the sorted, deduplicated candidate list (Eq. 8-9).
//   scan_kernel    full-history scores e_i = q.k_i/sqrt(d) (Eq. 4) for the KV heads that
//                  have at least one query head on the exact path; key rows stream once
//                  through the tensor cores for all G query heads of the group.
//   finish_kernel  one CTA per (sequence, query head): candidate scores (Eq. 10) or
//                  threshold collection from the scan, Top-K (Eq. 1 / Eq. 11), softmax.V
//                  over the winners (Eq. 12), support insert.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

namespace retopk {

constexpr int PATH_REUSE = 0, PATH_FALLBACK = 1, PATH_REFRESH = 2;
constexpr int MODE_RETOPK = 0, MODE_EXACT = 1;

constexpr int RECALL_THREADS = 256;
constexpr int SCAN_THREADS = 256;
constexpr int FINISH_THREADS = 512;
constexpr int SAMPLE_MAX = 8192;     // scores sampled to place the collection threshold
constexpr int SAMPLE_BINS = 2048;    // histogram over the top 11 bits of the score key
constexpr int NS_MIN = 4096;         // smallest candidate capacity of finish_kernel

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
    int NS;                  // candidate capacity (entries) of finish_kernel's shared lists
    int rows_per_cta;        // key rows per scan CTA (multiple of 128)
    const uint16_t* q;
    const uint16_t* k;
    const uint16_t* v;
    uint16_t* out;
    float* qbar_cache;       // [B*Hq][M][d]
    int32_t* sup_cache;      // [B*Hq][M][K]
    uint8_t* ws_path;        // [B*Hq]
    float* ws_rho;           // [B*Hq]
    int32_t* ws_ncand;       // [B*Hq]
    int32_t* ws_cand;        // [B*Hq][cap]
    float* ws_scores;        // [B*Hq][score_stride]
    long long* counters;     // [B*Hq][4] reuse, fallback, refresh, cand_sum
    unsigned int* status;
    unsigned long long* slow_select;
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
// recall_kernel
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(RECALL_THREADS) recall_kernel(const StepArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* s_q = reinterpret_cast<float*>(smem_raw);           // [d] normalised query
    float* s_rho = s_q + a.d;                                    // [M]
    int* s_sel = reinterpret_cast<int*>(s_rho + a.M);            // [r]
    int* s_ws = s_sel + a.r;                                     // [8]
    float* s_misc = reinterpret_cast<float*>(s_ws + 8);          // [4]
    const int head_words = a.d + a.M + a.r + 8 + 4;
    uint32_t* s_bm = reinterpret_cast<uint32_t*>(smem_raw) + ((head_words + 3) & ~3);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bh = blockIdx.x;
    const int d = a.d, M = a.M, fill = a.fill;

    // normalised query (text above Eq. 6)
    if (warp == 0) {
        const uint16_t* qrow = a.q + (size_t)bh * d;
        float x[4], acc = 0.f;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            int j = lane + 32 * u;
            x[u] = (j < d) ? __uint_as_float((uint32_t)qrow[j] << 16) : 0.f;
            acc = fmaf(x[u], x[u], acc);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        const float nrm = sqrtf(acc);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            int j = lane + 32 * u;
            if (j < d) s_q[j] = nrm > 0.f ? x[u] / nrm : 0.f;
        }
    }
    __syncthreads();

    // Eq. 6: rho_c for every cached entry
    for (int c = warp; c < fill; c += RECALL_THREADS / 32) {
        const float4* row = reinterpret_cast<const float4*>(a.qbar_cache + ((size_t)bh * M + c) * d);
        float acc = 0.f;
        for (int j = lane; j < d / 4; j += 32) {
            float4 x = row[j];
            acc = fmaf(x.x, s_q[4 * j], acc);
            acc = fmaf(x.y, s_q[4 * j + 1], acc);
            acc = fmaf(x.z, s_q[4 * j + 2], acc);
            acc = fmaf(x.w, s_q[4 * j + 3], acc);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) s_rho[c] = acc;
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
        if (lane == 0) s_misc[0] = rho_max;
    }
    __syncthreads();
    const float rho_max = s_misc[0];

    // Eq. 13
    int path;
    if (a.refresh) path = PATH_REFRESH;
    else if (rho_max < a.tau) path = PATH_FALLBACK;
    else path = PATH_REUSE;

    // insert the normalised query now: every similarity of this step has been taken
    for (int j = tid; j < d; j += RECALL_THREADS)
        a.qbar_cache[((size_t)bh * M + a.slot) * d + j] = s_q[j];

    int n_cand = a.L;
    if (path == PATH_REUSE) {
        // Eq. 8-9: bitmap over key positions, then ordered extraction = sorted unique list
        const int L = a.L;
        const int nwords = (L + 31) >> 5;
        for (int w = tid; w < nwords; w += RECALL_THREADS) s_bm[w] = 0u;
        __syncthreads();
        bool bad = false;
        for (int s = 0; s < n_sel; ++s) {
            const int c = s_sel[s];
            if (c < 0) continue;
            const int32_t* sp = a.sup_cache + ((size_t)bh * M + c) * a.K;
            for (int i = tid; i < a.K; i += RECALL_THREADS) {
                const int idx = sp[i];
                if (idx >= 0) {
                    if (idx < L) atomicOr(&s_bm[idx >> 5], 1u << (idx & 31));
                    else bad = true;
                }
            }
        }
        const int w_lo = L - a.W > 0 ? L - a.W : 0;
        for (int i = w_lo + tid; i < L; i += RECALL_THREADS) atomicOr(&s_bm[i >> 5], 1u << (i & 31));
        if (bad) atomicOr(a.status, 1u);
        __syncthreads();
        const int wpt = (nwords + RECALL_THREADS - 1) / RECALL_THREADS;
        const int w0 = tid * wpt;
        const int w1 = (w0 + wpt < nwords) ? w0 + wpt : nwords;
        int cnt = 0;
        for (int w = w0; w < w1; ++w) cnt += __popc(s_bm[w]);
        int total;
        int pos = block_excl_scan<RECALL_THREADS>(cnt, s_ws, total);
        int32_t* cand = a.ws_cand + (size_t)bh * a.cap;
        for (int w = w0; w < w1; ++w) {
            uint32_t bits = s_bm[w];
            while (bits) {
                const int b = __ffs(bits) - 1;
                cand[pos++] = w * 32 + b;
                bits &= bits - 1;
            }
        }
        n_cand = total;
    }

    if (tid == 0) {
        a.ws_path[bh] = (uint8_t)path;
        a.ws_rho[bh] = rho_max;
        a.ws_ncand[bh] = n_cand;
        long long* cnt = a.counters + (size_t)bh * 4;
        cnt[path] += 1;
        if (path == PATH_REUSE) cnt[3] += n_cand;
    }
}

// ------------------------------------------------------------------------------------
// scan_kernel: full-history scores on the tensor cores (mma.sync m16n8k16, bf16 -> fp32)
//
// A 16-row key tile is the A operand, the group's query heads (zero padded to 8) the B
// operand.  A dot product does not care in which order its terms are paired, so each
// thread loads 16 contiguous bytes of a key row straight into its A-fragment registers
// and the query fragment is permuted to match: no shared memory, no transposes.
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
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int bkv = blockIdx.y;                 // b * Hkv + kv head
    const int b = bkv / a.Hkv, kvh = bkv % a.Hkv;
    const int G = a.G, L = a.L;
    const int head0 = b * a.Hq + kvh * G;       // first query head of the group

    // which heads of the group want full scores this step
    unsigned need = 0;
    if (a.mode == MODE_EXACT) need = (1u << G) - 1u;
    else
        for (int j = 0; j < G; ++j)
            if (a.ws_path[head0 + j] != PATH_REUSE) need |= 1u << j;
    if (need == 0) return;

    const int row_begin = blockIdx.x * a.rows_per_cta;
    if (row_begin >= L) return;
    const int row_end = (row_begin + a.rows_per_cta < L) ? row_begin + a.rows_per_cta : L;

    // query fragments (B operand), permuted like the key loads below
    uint32_t bq[NTILE][NJ][2][2];
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

    const uint16_t* kbase = a.k + (size_t)bkv * a.max_seq_len * D;
    const float scale = a.scale;

    for (int tile = row_begin + warp * 16; tile < row_end; tile += (SCAN_THREADS / 32) * 16) {
        int r0 = tile + g, r1 = tile + g + 8;
        const int c0 = r0 < L ? r0 : L - 1, c1 = r1 < L ? r1 : L - 1;   // clamp, never read past L
        const uint16_t* p0 = kbase + (size_t)c0 * D + t * 8;
        const uint16_t* p1 = kbase + (size_t)c1 * D + t * 8;
        uint4 x[NJ], y[NJ];
#pragma unroll
        for (int j = 0; j < NJ; ++j) {
            x[j] = ldg_stream(p0 + j * 32);
            y[j] = ldg_stream(p1 + j * 32);
        }
#pragma unroll
        for (int nt = 0; nt < NTILE; ++nt) {
            float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
                mma_bf16_16816(c, x[j].x, y[j].x, x[j].y, y[j].y, bq[nt][j][0][0], bq[nt][j][0][1]);
                mma_bf16_16816(c, x[j].z, y[j].z, x[j].w, y[j].w, bq[nt][j][1][0], bq[nt][j][1][1]);
            }
            // c0,c1: row r0, heads 2t, 2t+1 of this tile; c2,c3: row r1
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int head = nt * 8 + 2 * t + e;
                if (head < G && ((need >> head) & 1u)) {
                    float* srow = a.ws_scores + (size_t)(head0 + head) * a.score_stride;
                    if (r0 < row_end) srow[r0] = c[e] * scale;
                    if (r1 < row_end) srow[r1] = c[2 + e] * scale;
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------
// selection primitives shared by both paths of finish_kernel
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

// ------------------------------------------------------------------------------------
// finish_kernel
// ------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(FINISH_THREADS) finish_kernel(const StepArgs a) {
    constexpr int NT = FINISH_THREADS;
    constexpr int LPR = D / 8;                  // lanes per bf16 row (16 bytes each)
    constexpr int RPW = 32 / LPR;               // rows per warp load
    constexpr int SLOTS = (NT / 32) * RPW;      // rows per block load
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint32_t* s_key = reinterpret_cast<uint32_t*>(smem_raw);        // [NS]
    int32_t* s_idx = reinterpret_cast<int32_t*>(s_key + a.NS);      // [NS]
    int32_t* s_sup_idx = s_idx + a.NS;                              // [K]
    uint32_t* s_sup_key = reinterpret_cast<uint32_t*>(s_sup_idx + a.K);   // [K]
    float* s_w = reinterpret_cast<float*>(s_sup_key + a.K);         // [K]
    uint32_t* s_hist = reinterpret_cast<uint32_t*>(s_w + a.K);      // [SAMPLE_BINS]
    int* s_ws = reinterpret_cast<int*>(s_hist + SAMPLE_BINS);       // [32]
    int* s_misc = s_ws + 32;                                        // [8]
    float* s_red = reinterpret_cast<float*>(smem_raw);              // [SLOTS][D], aliases s_key

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LPR, myslot = warp * RPW + lane / LPR;
    const int bh = blockIdx.x;
    const int b = bh / a.Hq, h = bh % a.Hq;
    const int bkv = b * a.Hkv + h / a.G;
    const int K = a.K, L = a.L, NS = a.NS;
    const int path = (a.mode == MODE_EXACT) ? PATH_FALLBACK : (int)a.ws_path[bh];
    const uint16_t* kbase = a.k + (size_t)bkv * a.max_seq_len * D;
    const uint16_t* vbase = a.v + (size_t)bkv * a.max_seq_len * D;

    int n = 0;        // entries in s_key / s_idx
    int ns = -1;      // selected entries in s_sup_*; -1 = not selected yet

    if (path == PATH_REUSE) {
        // Eq. 10: exact current-query scores on the candidate rows only
        n = a.ws_ncand[bh];
        const int32_t* cand = a.ws_cand + (size_t)bh * a.cap;
        for (int i = tid; i < n; i += NT) s_idx[i] = cand[i];
        float qf[8];
        unpack8(*reinterpret_cast<const uint4*>(a.q + (size_t)bh * D + sub * 8), qf);
        __syncthreads();
        for (int base = 0; base < n; base += SLOTS * 4) {
            uint4 x[4];
            int ii[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                ii[u] = base + u * SLOTS + myslot;
                const int idx = ii[u] < n ? s_idx[ii[u]] : 0;
                x[u] = ii[u] < n ? ldg_stream(kbase + (size_t)idx * D + sub * 8) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float acc = dot8(x[u], qf);
#pragma unroll
                for (int o = LPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
                if (sub == 0 && ii[u] < n) s_key[ii[u]] = score_key(acc * a.scale);
            }
        }
        __syncthreads();
    } else {
        // Eq. 1 on the scores written by scan_kernel
        const float* sc = a.ws_scores + (size_t)bh * a.score_stride;
        bool slow = false;
        if (L <= K) {
            slow = false;
            for (int i = tid; i < L; i += NT) { s_sup_idx[i] = i; s_sup_key[i] = score_key(sc[i]); }
            ns = L;
            __syncthreads();
        } else {
            // 1. place a threshold from a block-strided sample so that about 2K scores pass
            const bool all = L <= SAMPLE_MAX;
            const int n_s = all ? L : SAMPLE_MAX;
            for (int i = tid; i < SAMPLE_BINS; i += NT) s_hist[i] = 0;
            __syncthreads();
            const int blk = L >> 3;
            for (int i = tid; i < n_s; i += NT) {
                const int pos = all ? i : (i >> 10) * blk + (i & 1023);
                atomicAdd(&s_hist[score_key(sc[pos]) >> 21], 1u);
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
                int c = 0;
#pragma unroll
                for (int u = 0; u < SAMPLE_BINS / NT; ++u)
                    c += (int)s_hist[SAMPLE_BINS - 1 - (SAMPLE_BINS / NT) * tid - u];
                int total;
                const int above = block_excl_scan<NT>(c, s_ws, total);
                if (above < j && j <= above + c) {
                    int acc = above;
                    for (int u = 0; u < SAMPLE_BINS / NT; ++u) {
                        const int bin = SAMPLE_BINS - 1 - (SAMPLE_BINS / NT) * tid - u;
                        acc += (int)s_hist[bin];
                        if (acc >= j) { s_misc[2] = bin; break; }
                    }
                }
                __syncthreads();
                thr_key = (uint32_t)s_misc[2] << 21;
            }
            // 2. ordered collection of every score at or above the threshold
            int run = 0;
            for (int base = 0; base < L; base += NT * 4) {
                const int i0 = base + tid * 4;
                uint32_t key[4];
                int f[4], cnt = 0;
                if (i0 < L) {
                    const float4 x = *reinterpret_cast<const float4*>(sc + i0);
                    key[0] = score_key(x.x); key[1] = score_key(x.y);
                    key[2] = score_key(x.z); key[3] = score_key(x.w);
#pragma unroll
                    for (int u = 0; u < 4; ++u) { f[u] = (i0 + u < L) && key[u] >= thr_key; cnt += f[u]; }
                } else {
#pragma unroll
                    for (int u = 0; u < 4; ++u) { f[u] = 0; key[u] = 0; }
                }
                int total;
                int pos = run + block_excl_scan<NT>(cnt, s_ws, total);
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (f[u]) {
                        if (pos < NS) { s_key[pos] = key[u]; s_idx[pos] = i0 + u; }
                        ++pos;
                    }
                run += total;
            }
            __syncthreads();
            n = run;
            if (n > NS || n < K) slow = true;
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
    }

    if (ns < 0) {
        // Eq. 11 / Eq. 1: Top-K of the n listed entries
        SmemSrc src{s_key, s_idx};
        if (n <= K) {
            for (int i = tid; i < n; i += NT) { s_sup_idx[i] = s_idx[i]; s_sup_key[i] = s_key[i]; }
            ns = n;
        } else {
            uint32_t vstar;
            int need_eq;
            radix_select<NT>(src, n, K, s_hist, s_misc, vstar, need_eq);
            ordered_emit<NT>(src, n, vstar, need_eq, s_sup_idx, s_sup_key, s_ws);
            ns = K;
        }
        __syncthreads();
    }

    // record the support (cache insert / caller's index output)
    int32_t* sup_out = nullptr;
    if (a.mode == MODE_RETOPK) sup_out = a.sup_cache + ((size_t)bh * a.M + a.slot) * K;
    else if (a.idx_out) sup_out = a.idx_out + (size_t)bh * K;
    if (sup_out)
        for (int i = tid; i < K; i += NT) sup_out[i] = i < ns ? s_sup_idx[i] : -1;

    // Eq. 12: softmax over the selected scores, then the weighted value rows
    uint32_t kmax = 0;
    for (int i = tid; i < ns; i += NT) kmax = max(kmax, s_sup_key[i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
    if (lane == 0) s_ws[warp] = (int)kmax;
    __syncthreads();
    kmax = 0;
    for (int w = 0; w < NT / 32; ++w) kmax = max(kmax, (uint32_t)s_ws[w]);
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
    for (int w = 0; w < NT / 32; ++w) denom += s_wsf[w];

    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    for (int base = 0; base < ns; base += SLOTS * 4) {
        uint4 x[4];
        float w[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = base + u * SLOTS + myslot;
            const bool ok = i < ns;
            w[u] = ok ? s_w[i] : 0.f;
            x[u] = ok ? ldg_stream(vbase + (size_t)s_sup_idx[i] * D + sub * 8) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            float f[8];
            unpack8(x[u], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = fmaf(w[u], f[e], acc[e]);
        }
    }
    __syncthreads();   // s_key (aliased by s_red) is no longer read
#pragma unroll
    for (int e = 0; e < 8; ++e) s_red[myslot * D + sub * 8 + e] = acc[e];
    __syncthreads();
    for (int j = tid; j < D; j += NT) {
        float sum = 0.f;
        for (int s = 0; s < SLOTS; ++s) sum += s_red[s * D + j];
        const float o = ns > 0 ? sum / denom : 0.f;
        a.out[(size_t)bh * D + j] = __bfloat16_as_ushort(__float2bfloat16_rn(o));
    }
}

// Clear the caches (supports to -1, queries and counters to 0).
__global__ void reset_kernel(float* qbar, size_t n_q, int32_t* sup, size_t n_sup, long long* counters,
                             size_t n_cnt, unsigned int* status, unsigned long long* slow) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t t0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (size_t i = t0; i < n_q; i += stride) qbar[i] = 0.f;
    for (size_t i = t0; i < n_sup; i += stride) sup[i] = -1;
    for (size_t i = t0; i < n_cnt; i += stride) counters[i] = 0;
    if (t0 == 0) { *status = 0u; *slow = 0ull; }
}

}  // namespace retopk
