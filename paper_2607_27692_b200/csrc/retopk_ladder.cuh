// Less fused forms of the reuse path, for measuring what each fusion step buys (Table 4 of
// the paper reports such a ladder for its own kernels; the cut points below are this
// library's, chosen to follow the paper's description of its five stages).
//
//   level 1  separate kernels: similarity | top-r + decision | candidate union | pack the
//            candidate key rows | score the packed rows | top-K | softmax.V | cache insert
//   level 2  cache search fused with the support union (one "discover" kernel); candidate
//            rows scored in place through their indices (no packing)
//   level 3  selection, sparse output and cache update fused into one kernel
//   level 4  as level 3, with the intermediate buffers kept by the context instead of being
//            allocated from a stream-ordered pool in every step (a host-side difference)
//   level 5  candidate construction through output in one kernel: recall_kernel +
//            finish_kernel, the production path
//
// Every level runs the same device functions on the same lanes as the production path, so
// supports and outputs are bit-identical across levels.  Heads on the exact path are served
// by scan_kernel + finish_kernel at every level.  One block of LADDER_THREADS per head.
#pragma once

#include "retopk_kernels.cuh"

namespace retopk {

constexpr int LADDER_THREADS = 1024;

// ---- level 1 --------------------------------------------------------------------------

// Eq. 6 alone: similarities and the normalised query to global memory.
template <int D>
__global__ void __launch_bounds__(LADDER_THREADS, 1) ladder_similarity_kernel(const StepArgs a) {
    constexpr int NT = LADDER_THREADS;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // layout (words): q[D] rho[M + 3]
    float* s_q = reinterpret_cast<float*>(smem_raw);
    float* s_rho = s_q + D;
    const int tid = threadIdx.x, bh = blockIdx.x;
    cache_similarities<D, NT>(a, bh, s_q, s_rho);
    __syncthreads();
    for (int c = tid; c < a.fill; c += NT) a.lw_rho[(size_t)bh * a.M + c] = s_rho[c];
    if (tid < D) a.lw_qbar[(size_t)bh * D + tid] = s_q[tid];
}

// Eq. 7 and Eq. 13 from the stored similarities.
__global__ void __launch_bounds__(LADDER_THREADS, 1) ladder_topr_kernel(const StepArgs a) {
    constexpr int NT = LADDER_THREADS;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // layout (words): rho[M + 3] ws[WS_WORDS] sel[r] misc[4]
    float* s_rho = reinterpret_cast<float*>(smem_raw);
    int* s_ws = reinterpret_cast<int*>(s_rho + ((a.M + 3) & ~3));
    int* s_sel = s_ws + WS_WORDS;
    float* s_misc = reinterpret_cast<float*>(s_sel + a.r);
    const int tid = threadIdx.x, bh = blockIdx.x;
    if (tid < a.r) s_sel[tid] = -1;
    if (tid == 0) s_misc[0] = -CUDART_INF_F;
    for (int c = tid; c < a.fill; c += NT) s_rho[c] = a.lw_rho[(size_t)bh * a.M + c];
    __syncthreads();
    int sel8[8];
    const float rho_max = recall_slots<NT>(a, s_rho, s_sel, s_misc, s_ws, sel8);
    record_decision(a, bh, kv_group_of(bh, a), s_sel, decide_path(a, rho_max), rho_max);
}

// Shared-memory carve-up of the union: sel[r] ws[WS_WORDS] | idx[cap] | bitmap
struct UnionSmem {
    int* sel;
    int* ws;
    int32_t* idx;
    uint32_t* bm;
};
__device__ __forceinline__ UnionSmem union_smem(const StepArgs& a, unsigned char* base) {
    UnionSmem u;
    u.sel = reinterpret_cast<int*>(base);
    u.ws = u.sel + ((a.r + 3) & ~3);
    u.idx = u.ws + WS_WORDS;
    u.bm = reinterpret_cast<uint32_t*>(u.idx + ((a.cap + 3) & ~3));
    return u;
}

// Eq. 8-9 for a head whose recalled slots are in u.sel: list to global memory.
template <int NT>
__device__ __forceinline__ void union_to_global(const StepArgs& a, int bh, const UnionSmem& u) {
    const int tid = threadIdx.x;
    const int n_sel = a.r < a.fill ? a.r : a.fill;
    {
        const int nwords = (a.L + 31) >> 5;
        uint4* bm4 = reinterpret_cast<uint4*>(u.bm);
        for (int w = tid; w < (nwords + 3) >> 2; w += NT) bm4[w] = make_uint4(0, 0, 0, 0);
    }
    __syncthreads();
    const int n = candidate_union<NT>(a, bh, u.sel, n_sel, u.bm, u.idx, u.ws);
    __syncthreads();
    for (int i = tid; i < n; i += NT) a.lw_cand[(size_t)bh * a.cap + i] = u.idx[i];
    if (a.dbg_cand)
        for (int i = tid; i < n; i += NT) a.dbg_cand[(size_t)bh * a.cap + i] = u.idx[i];
    if (tid == 0) a.ws_ncand[bh] = n;
}

__global__ void __launch_bounds__(LADDER_THREADS, 1) ladder_union_kernel(const StepArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, bh = blockIdx.x;
    if (a.ws_path[bh] != PATH_REUSE) return;
    const UnionSmem u = union_smem(a, smem_raw);
    if (tid < a.r) u.sel[tid] = a.ws_sel[(size_t)bh * a.r + tid];
    union_to_global<LADDER_THREADS>(a, bh, u);
}

// Copy the candidate key rows of a head into a packed buffer (16 bytes per thread and trip).
template <int D>
__global__ void __launch_bounds__(LADDER_THREADS, 1) ladder_pack_rows_kernel(const StepArgs a) {
    constexpr int LPR = D / 8;
    const int tid = threadIdx.x, bh = blockIdx.x;
    if (a.ws_path[bh] != PATH_REUSE) return;
    const int n = a.ws_ncand[bh];
    const uint4* src = reinterpret_cast<const uint4*>(a.k + (size_t)kv_group_of(bh, a) * a.max_seq_len * D);
    uint4* dst = reinterpret_cast<uint4*>(a.lw_rows + (size_t)bh * a.cap * D);
    const int32_t* cand = a.lw_cand + (size_t)bh * a.cap;
    for (int p = tid; p < n * LPR; p += LADDER_THREADS)
        dst[p] = src[(size_t)cand[p / LPR] * LPR + p % LPR];
}

// Eq. 10 as a kernel of its own: rows through their indices (INDEXED) or from the packed
// buffer of level 1; score keys to global memory.
template <int D, bool INDEXED>
__global__ void __launch_bounds__(LADDER_THREADS, 1) ladder_score_kernel(const StepArgs a) {
    constexpr int NT = LADDER_THREADS;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // layout (words): qraw[D] idx[cap] | stage[depth*NT*4]
    float* s_qraw = reinterpret_cast<float*>(smem_raw);
    int32_t* s_idx = reinterpret_cast<int32_t*>(s_qraw + D);
    uint4* s_stage = reinterpret_cast<uint4*>(s_idx + ((a.cap + 3) & ~3));
    const int tid = threadIdx.x, bh = blockIdx.x;
    if (a.ws_path[bh] != PATH_REUSE) return;
    const int n = a.ws_ncand[bh];
    if (tid < D / 2) {
        const uint32_t raw = reinterpret_cast<const uint32_t*>(a.q + (size_t)bh * D)[tid];
        s_qraw[2 * tid] = bf16_lo(raw);
        s_qraw[2 * tid + 1] = bf16_hi(raw);
    }
    if (INDEXED)
        for (int i = tid; i < n; i += NT) s_idx[i] = a.lw_cand[(size_t)bh * a.cap + i];
    __syncthreads();
    const uint16_t* rows = INDEXED ? a.k + (size_t)kv_group_of(bh, a) * a.max_seq_len * D
                                   : a.lw_rows + (size_t)bh * a.cap * D;
    score_candidates<D, NT, INDEXED>(rows, s_idx, n, s_qraw, s_stage, a.stage_depth, a.scale,
                                     a.lw_key + (size_t)bh * a.cap);
}

// Eq. 11 as a kernel of its own.
__global__ void __launch_bounds__(LADDER_THREADS, 1) ladder_select_kernel(const StepArgs a) {
    constexpr int NT = LADDER_THREADS;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // layout (words): ws[WS_WORDS] hist[SCRATCH_WORDS] sup_idx[K] sup_key[K] idx[cap] key[cap]
    int* s_ws = reinterpret_cast<int*>(smem_raw);
    uint32_t* s_hist = reinterpret_cast<uint32_t*>(s_ws + WS_WORDS);
    int32_t* s_sup_idx = reinterpret_cast<int32_t*>(s_hist + SCRATCH_WORDS);
    uint32_t* s_sup_key = reinterpret_cast<uint32_t*>(s_sup_idx + a.K);
    int32_t* s_idx = reinterpret_cast<int32_t*>(s_sup_key + a.K);
    uint32_t* s_key = reinterpret_cast<uint32_t*>(s_idx + a.cap);
    const int tid = threadIdx.x, bh = blockIdx.x;
    if (a.ws_path[bh] != PATH_REUSE) return;
    const int n = a.ws_ncand[bh];
    for (int i = tid; i < n; i += NT) {
        s_idx[i] = a.lw_cand[(size_t)bh * a.cap + i];
        s_key[i] = a.lw_key[(size_t)bh * a.cap + i];
    }
    __syncthreads();
    uint32_t kmax;
    const int ns = select_listed<NT>(s_key, s_idx, n, a.K, s_sup_idx, s_sup_key, s_hist, s_ws, &kmax);
    for (int i = tid; i < ns; i += NT) {
        a.lw_sup_idx[(size_t)bh * a.K + i] = s_sup_idx[i];
        a.lw_sup_key[(size_t)bh * a.K + i] = s_sup_key[i];
    }
    if (tid == 0) {
        a.lw_meta[bh * 4 + 0] = ns;
        a.lw_meta[bh * 4 + 1] = (int32_t)kmax;
        a.lw_meta[bh * 4 + 2] = 1;
    }
}

// Eq. 12 as a kernel of its own.
template <int D>
__global__ void __launch_bounds__(LADDER_THREADS, 1) ladder_attend_kernel(const StepArgs a) {
    constexpr int NT = LADDER_THREADS, NW = NT / 32;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // layout (words): ws[WS_WORDS] sup_idx[K] sup_key[K] w[K] red[NW*D+NT] | stage[depth*NT*4]
    int* s_ws = reinterpret_cast<int*>(smem_raw);
    int32_t* s_sup_idx = reinterpret_cast<int32_t*>(s_ws + WS_WORDS);
    uint32_t* s_sup_key = reinterpret_cast<uint32_t*>(s_sup_idx + a.K);
    float* s_w = reinterpret_cast<float*>(s_sup_key + a.K);
    float* s_red = reinterpret_cast<float*>(s_ws + WS_WORDS + ((3 * a.K + 3) & ~3));
    uint4* s_stage = reinterpret_cast<uint4*>(s_red + NW * D + NT);
    const int tid = threadIdx.x, bh = blockIdx.x;
    if (a.ws_path[bh] != PATH_REUSE) return;
    const int ns = a.lw_meta[bh * 4 + 0];
    const uint32_t kmax = (uint32_t)a.lw_meta[bh * 4 + 1];
    for (int i = tid; i < ns; i += NT) {
        s_sup_idx[i] = a.lw_sup_idx[(size_t)bh * a.K + i];
        s_sup_key[i] = a.lw_sup_key[(size_t)bh * a.K + i];
    }
    __syncthreads();
    attend<D, NT>(a.v + (size_t)kv_group_of(bh, a) * a.max_seq_len * D, ns, s_sup_idx, s_sup_key, s_w, s_red, s_ws,
                  s_stage, a.stage_depth, kmax, a.out + (size_t)bh * D);
    if (tid == 0) {
        const int n = a.ws_ncand[bh];
        atomicAdd(a.counters + (size_t)bh * 4 + PATH_REUSE, 1ull);
        atomicAdd(a.counters + (size_t)bh * 4 + 3, (unsigned long long)n);
    }
}

// Cache update as a kernel of its own: the support of a head on the reuse path (-1 padded)
// and, with insert_q, the normalised query of every head.
__global__ void __launch_bounds__(LADDER_THREADS, 1) ladder_insert_kernel(const StepArgs a, int insert_q) {
    const int tid = threadIdx.x, bh = blockIdx.x;
    if (insert_q && tid < a.d)
        store_qbar(a, ((size_t)bh * a.M + a.slot) * a.d + tid, a.lw_qbar[(size_t)bh * a.d + tid]);
    if (a.ws_path[bh] != PATH_REUSE) return;
    const int ns = a.lw_meta[bh * 4 + 0];
    int32_t* sup_out = a.sup_cache + ((size_t)bh * a.M + a.slot) * a.K;
    for (int i = tid; i < a.K; i += LADDER_THREADS) sup_out[i] = i < ns ? a.lw_sup_idx[(size_t)bh * a.K + i] : -1;
}

// ---- level 2 --------------------------------------------------------------------------

// Cache search and support union in one kernel: the recall stage, then Eq. 8-9 for a
// head that stays on the reuse path.
template <int D>
__global__ void __launch_bounds__(LADDER_THREADS, 1) ladder_discover_kernel(const StepArgs a) {
    constexpr int NT = LADDER_THREADS;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // layout (words): q[D] rho[M + 3] misc[4] | union carve-up (its sel[] is the recall's)
    float* s_q = reinterpret_cast<float*>(smem_raw);
    float* s_rho = s_q + D;
    float* s_misc = s_rho + ((a.M + 3) & ~3);
    const UnionSmem u = union_smem(a, reinterpret_cast<unsigned char*>(s_misc + 4));
    const int tid = threadIdx.x, bh = blockIdx.x;
    if (tid < a.r) u.sel[tid] = -1;
    if (tid == 0) s_misc[0] = -CUDART_INF_F;
    cache_similarities<D, NT>(a, bh, s_q, s_rho);
    __syncthreads();
    int sel8[8];
    const float rho_max = recall_slots<NT>(a, s_rho, u.sel, s_misc, u.ws, sel8);
    const int path = decide_path(a, rho_max);
    if (tid < D) store_qbar(a, ((size_t)bh * a.M + a.slot) * D + tid, s_q[tid]);
    record_decision(a, bh, kv_group_of(bh, a), u.sel, path, rho_max);
    if (path == PATH_REUSE) union_to_global<NT>(a, bh, u);
}

// ---- level 3 --------------------------------------------------------------------------

// Eq. 11, Eq. 12 and the support insert in one kernel, from the stored candidate scores.
template <int D>
__global__ void __launch_bounds__(LADDER_THREADS, 1) ladder_select_attend_insert_kernel(const StepArgs a) {
    constexpr int NT = LADDER_THREADS, NW = NT / 32;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // layout (words): ws[WS_WORDS] hist[SCRATCH_WORDS] sup_idx[K] sup_key[K] w[K]
    //                 | big: idx[cap] key[cap], aliased later by red[NW*D+NT] | stage[depth*NT*4]
    int* s_ws = reinterpret_cast<int*>(smem_raw);
    uint32_t* s_hist = reinterpret_cast<uint32_t*>(s_ws + WS_WORDS);
    int32_t* s_sup_idx = reinterpret_cast<int32_t*>(s_hist + SCRATCH_WORDS);
    uint32_t* s_sup_key = reinterpret_cast<uint32_t*>(s_sup_idx + a.K);
    float* s_w = reinterpret_cast<float*>(s_sup_key + a.K);
    const int head_words = (WS_WORDS + SCRATCH_WORDS + 3 * a.K + 3) & ~3;
    int32_t* s_idx = reinterpret_cast<int32_t*>(smem_raw) + head_words;
    uint32_t* s_key = reinterpret_cast<uint32_t*>(s_idx + a.cap);
    float* s_red = reinterpret_cast<float*>(s_idx);
    const int big_words = (max(2 * a.cap, NW * D + NT) + 3) & ~3;
    uint4* s_stage = reinterpret_cast<uint4*>(s_idx + big_words);
    const int tid = threadIdx.x, bh = blockIdx.x;
    if (a.ws_path[bh] != PATH_REUSE) return;
    const int n = a.ws_ncand[bh];
    for (int i = tid; i < n; i += NT) {
        s_idx[i] = a.lw_cand[(size_t)bh * a.cap + i];
        s_key[i] = a.lw_key[(size_t)bh * a.cap + i];
    }
    __syncthreads();
    uint32_t kmax;
    const int ns = select_listed<NT>(s_key, s_idx, n, a.K, s_sup_idx, s_sup_key, s_hist, s_ws, &kmax);
    int32_t* sup_out = a.sup_cache + ((size_t)bh * a.M + a.slot) * a.K;
    for (int i = tid; i < a.K; i += NT) sup_out[i] = i < ns ? s_sup_idx[i] : -1;
    attend<D, NT>(a.v + (size_t)kv_group_of(bh, a) * a.max_seq_len * D, ns, s_sup_idx, s_sup_key, s_w, s_red, s_ws,
                  s_stage, a.stage_depth, kmax, a.out + (size_t)bh * D);
    if (tid == 0) {
        atomicAdd(a.counters + (size_t)bh * 4 + PATH_REUSE, 1ull);
        atomicAdd(a.counters + (size_t)bh * 4 + 3, (unsigned long long)n);
    }
}

}  // namespace retopk
