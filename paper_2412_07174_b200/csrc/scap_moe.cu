// Mixture-of-experts FFN layer: routing (softmax, top-k, renormalise) is recomputed by every
// compaction CTA, the SwiGLU kernels run as one grouped launch with blockIdx.z = expert (experts
// without rows exit at once), and a small kernel forms the weighted sum in selection order.
#include <string.h>

#include "scap_fc.cuh"

namespace scap {

struct Route {  // device-resident routing table, written by the compaction kernel
    int nb[SCAP_MAX_EXPERTS];                         // rows routed to each expert
    int rows[SCAP_MAX_EXPERTS][SCAP_MAX_BATCH];       // their batch rows, ascending
    int slots[SCAP_MAX_EXPERTS][SCAP_MAX_BATCH];      // row * top_k + position in the row's selection
    float w[SCAP_MAX_BATCH][SCAP_MAX_TOP_K];          // renormalised weights, selection order
};

struct MoeArgs {
    scap_expert ex[SCAP_MAX_EXPERTS];
    int E, top_k, B, D, F;
    const void *h;
    const float *logits;
    unsigned char *ws;
    size_t group_bytes;  // workspace stride between experts
    FcLayout L1, L2;     // offsets inside one expert's workspace
    Route *route;
    float *yslot;        // [B * top_k, D]
    float *y;
    int *expert_out;
    float *weight_out;
};

// Routing for all rows, by one CTA, into shared memory.  Selection compares the logits themselves
// (softmax is monotonic), ties to the lower index; weights are computed in binary64.
__device__ void compute_route(const float *__restrict__ logits, int B, int E, int top_k, Route *r, int *sel /*[B][top_k]*/) {
    const int tid = threadIdx.x;
    if (tid < B) {
        const float *lg = logits + (size_t)tid * E;
        uint32_t used = 0;
        double p[SCAP_MAX_TOP_K];
        float mx = -INFINITY;
        for (int e = 0; e < E; ++e) mx = fmaxf(mx, lg[e]);
        double tot = 0.0;
        for (int j = 0; j < top_k; ++j) {
            int best = -1;
            for (int e = 0; e < E; ++e)
                if (!((used >> e) & 1u) && (best < 0 || lg[e] > lg[best])) best = e;
            used |= 1u << best;
            sel[tid * SCAP_MAX_TOP_K + j] = best;
            p[j] = exp((double)lg[best] - (double)mx);
            tot += p[j];
        }
        for (int j = 0; j < top_k; ++j) r->w[tid][j] = (float)(p[j] / tot);
    }
    __syncthreads();
    if (tid < E) {
        int n = 0;
        for (int b = 0; b < B; ++b)
            for (int j = 0; j < top_k; ++j)
                if (sel[b * SCAP_MAX_TOP_K + j] == tid) {
                    r->rows[tid][n] = b;
                    r->slots[tid][n] = b * top_k + j;
                    ++n;
                }
        r->nb[tid] = n;
    }
    __syncthreads();
}

// grid (chunks of D, E).  Centre + threshold of h over the rows routed to expert blockIdx.y.
template <typename XT>
__global__ void __launch_bounds__(CH) moe_compact_kernel(const MoeArgs a) {
    __shared__ Route s_route;
    __shared__ int s_sel[SCAP_MAX_BATCH * SCAP_MAX_TOP_K];
    __shared__ int s_wcount[CH / 32];
    griddep_wait();
    griddep_launch_dependents();
    compute_route(a.logits, a.B, a.E, a.top_k, &s_route, s_sel);
    const int e = blockIdx.y, tid = threadIdx.x;
    if (blockIdx.x == 0) {  // publish the table entry of this expert; expert 0's CTA also the per-row data
        if (tid == 0) a.route->nb[e] = s_route.nb[e];
        if (tid < SCAP_MAX_BATCH) {
            a.route->rows[e][tid] = s_route.rows[e][tid];
            a.route->slots[e][tid] = s_route.slots[e][tid];
        }
        if (e == 0 && tid < a.B)
            for (int j = 0; j < a.top_k; ++j) {
                a.route->w[tid][j] = s_route.w[tid][j];
                if (a.expert_out) a.expert_out[tid * a.top_k + j] = s_sel[tid * SCAP_MAX_TOP_K + j];
                if (a.weight_out) a.weight_out[tid * a.top_k + j] = s_route.w[tid][j];
            }
    }
    const int nb = s_route.nb[e];
    if (nb == 0) return;
    unsigned char *w = a.ws + (size_t)e * a.group_bytes;
    int *tickets = reinterpret_cast<int *>(w + a.L1.tickets);
    const int gtid = blockIdx.x * CH + tid;
    for (int i = gtid; i < a.L1.tiles; i += gridDim.x * CH) tickets[i] = 0;
    const float tau = __ldg(a.ex[e].tau1);
    float d[SCAP_MAX_BATCH];
    uint32_t keepmask = 0;
    if (gtid < a.D)
        keepmask = centre_threshold<XT>(reinterpret_cast<const XT *>(a.h), (size_t)a.D, s_route.rows[e], a.ex[e].m1, tau, nb, gtid, d);
    compact_chunk((uint32_t)gtid, d, keepmask, nb, blockIdx.x, reinterpret_cast<int *>(w + a.L1.counts),
                  reinterpret_cast<uint32_t *>(w + a.L1.idx_local), reinterpret_cast<float *>(w + a.L1.xs_local), a.L1.Kpad,
                  s_wcount);
}

__device__ __forceinline__ void bind_layout_dev(GemvArgs &g, const FcLayout &L, unsigned char *w) {
    g.S = L.S;
    g.counts = reinterpret_cast<const int *>(w + L.counts);
    g.idx_local = reinterpret_cast<const uint32_t *>(w + L.idx_local);
    g.xs_local = reinterpret_cast<const float *>(w + L.xs_local);
    g.Kpad = L.Kpad;
    g.nchunks = L.nchunks;
    g.partials = reinterpret_cast<float *>(w + L.partials);
    g.tickets = reinterpret_cast<int *>(w + L.tickets);
}

// grid (tiles, S, E).  STAGE 1: packed gate|up GEMV with the z + compaction epilogue; STAGE 2: down GEMV
// writing each row to its (row, selection position) slot.
template <bool BF16, int BT, int STAGE>
__global__ void __launch_bounds__(GEMV_THREADS, gemv_min_blocks(BT)) moe_gemv_kernel(const MoeArgs a) {
    griddep_wait();
    griddep_launch_dependents();
    const int e = blockIdx.z;
    const int nb = __ldcg(&a.route->nb[e]);
    if (nb == 0) return;
    unsigned char *w = a.ws + (size_t)e * a.group_bytes;
    GemvArgs g = {};
    g.B = nb;
    if constexpr (STAGE == 1) {
        g.W = a.ex[e].Wgu; g.K = a.D; g.ldw = 2 * a.F; g.halves = 2; g.Nh = a.F;
        bind_layout_dev(g, a.L1, w);
        g.bias = a.ex[e].bgu_fused;
        g.m2 = a.ex[e].m2; g.tau2 = a.ex[e].tau2;
        g.counts2 = reinterpret_cast<int *>(w + a.L2.counts);
        g.idx_local2 = reinterpret_cast<uint32_t *>(w + a.L2.idx_local);
        g.xs_local2 = reinterpret_cast<float *>(w + a.L2.xs_local);
        g.Kpad2 = a.L2.Kpad;
        g.tickets_next = reinterpret_cast<int *>(w + a.L2.tickets);
        g.ntickets_next = a.L2.tiles;
        gemv_body<BF16, BT, MODE_GATHER, float, EPI_GLU>(g, blockIdx.x, blockIdx.y);
    } else {
        g.W = a.ex[e].Wd; g.K = a.F; g.ldw = a.D; g.halves = 1; g.Nh = a.D;
        bind_layout_dev(g, a.L2, w);
        g.bias = a.ex[e].bd_fused;
        g.y = a.yslot;
        g.out_rows = a.route->slots[e];
        gemv_body<BF16, BT, MODE_GATHER, float, EPI_BIAS>(g, blockIdx.x, blockIdx.y);
    }
}

// y[b, n] = sum_j w[b, j] * yslot[b * top_k + j, n], j ascending (selection order).
__global__ void __launch_bounds__(256) moe_combine_kernel(const MoeArgs a) {
    griddep_wait();
    griddep_launch_dependents();
    const int n = blockIdx.x * blockDim.x + threadIdx.x, b = blockIdx.y;
    if (n >= a.D) return;
    float acc = 0.0f;
    for (int j = 0; j < a.top_k; ++j)
        acc = fmaf(__ldcg(&a.route->w[b][j]), __ldcg(a.yslot + (size_t)(b * a.top_k + j) * a.D + n), acc);
    a.y[(size_t)b * a.D + n] = acc;
}

struct MoeLayout {
    FcLayout L1, L2;
    size_t group_bytes, route, yslot, total;
};

static MoeLayout moe_layout(int B, int D, int F, int E, int top_k) {
    MoeLayout M;
    M.L1 = fc_layout(B, D, 2 * F, 2, 0);
    M.L2 = fc_layout(B, F, D, 1, M.L1.total);
    M.group_bytes = align_up(M.L2.total, 256);
    size_t off = M.group_bytes * E;
    M.route = off;
    off = align_up(off + sizeof(Route), 256);
    M.yslot = off;
    off = align_up(off + sizeof(float) * (size_t)B * top_k * D, 256);
    M.total = off;
    return M;
}

template <bool BF16, int STAGE>
static cudaError_t launch_moe_gemv(const MoeArgs &a, int tiles, int S, cudaStream_t st) {
    const dim3 grid(tiles, S, a.E), block(GEMV_THREADS);
    const bool pdl = g_tune.pdl != 0;
    switch (batch_tile(a.B)) {
        case 1: return launch(moe_gemv_kernel<BF16, 1, STAGE>, grid, block, 0, st, pdl, a);
        case 2: return launch(moe_gemv_kernel<BF16, 2, STAGE>, grid, block, 0, st, pdl, a);
        case 4: return launch(moe_gemv_kernel<BF16, 4, STAGE>, grid, block, 0, st, pdl, a);
        case 8: return launch(moe_gemv_kernel<BF16, 8, STAGE>, grid, block, 0, st, pdl, a);
        default: return launch(moe_gemv_kernel<BF16, 16, STAGE>, grid, block, 0, st, pdl, a);
    }
}

}  // namespace scap

using namespace scap;

extern "C" {

size_t scap_moe_workspace(int B, int D, int F, int E, int top_k) {
    if (B < 1 || B > SCAP_MAX_BATCH || D < 1 || F < 1 || D > MAX_CHUNKS_SMEM * CH || F > MAX_CHUNKS_SMEM * CH || E < 1 ||
        E > SCAP_MAX_EXPERTS || top_k < 1 || top_k > SCAP_MAX_TOP_K || top_k > E)
        return 0;
    return moe_layout(B, D, F, E, top_k).total;
}

scap_status scap_moe_ffn(const void *h, const float *logits, const scap_expert *experts_host, int E, int top_k, float *y, int B,
                         int D, int F, scap_dtype dt, int *expert_out, float *weight_out, void *ws, size_t ws_bytes,
                         scap_stream_t stream) {
    if (!h || !logits || !experts_host || !y || !ws) return SCAP_ERR_INVALID_ARG;
    if (dt != SCAP_F16 && dt != SCAP_BF16) return SCAP_ERR_DTYPE;
    if (B < 1 || B > SCAP_MAX_BATCH || D < 1 || F < 1 || D > MAX_CHUNKS_SMEM * CH || F > MAX_CHUNKS_SMEM * CH || E < 1 ||
        E > SCAP_MAX_EXPERTS || top_k < 1 || top_k > SCAP_MAX_TOP_K || top_k > E)
        return SCAP_ERR_SHAPE;
    if (D % 8 != 0 || F % 8 != 0 || !aligned16(h) || !aligned16(y) || !aligned16(ws)) return SCAP_ERR_ALIGN;
    for (int e = 0; e < E; ++e) {
        const scap_expert &x = experts_host[e];
        if (!x.Wgu || !x.Wd || !x.tau1 || !x.tau2) return SCAP_ERR_INVALID_ARG;
        if (!aligned16(x.Wgu) || !aligned16(x.Wd) || (x.m1 && !aligned16(x.m1)) || (x.m2 && !aligned16(x.m2)) ||
            (x.bgu_fused && !aligned16(x.bgu_fused)) || (x.bd_fused && !aligned16(x.bd_fused)))
            return SCAP_ERR_ALIGN;
    }
    if (ws_bytes < scap_moe_workspace(B, D, F, E, top_k)) return SCAP_ERR_WORKSPACE;
    scap_status stt = check_device();
    if (stt != SCAP_OK) return stt;

    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const MoeLayout M = moe_layout(B, D, F, E, top_k);
    MoeArgs a;
    memset(&a, 0, sizeof(a));
    memcpy(a.ex, experts_host, sizeof(scap_expert) * E);
    a.E = E; a.top_k = top_k; a.B = B; a.D = D; a.F = F;
    a.h = h; a.logits = logits;
    a.ws = static_cast<unsigned char *>(ws);
    a.group_bytes = M.group_bytes;
    a.L1 = M.L1; a.L2 = M.L2;
    a.route = reinterpret_cast<Route *>(a.ws + M.route);
    a.yslot = reinterpret_cast<float *>(a.ws + M.yslot);
    a.y = y; a.expert_out = expert_out; a.weight_out = weight_out;
    const bool bf16 = dt == SCAP_BF16, pdl = g_tune.pdl != 0;

    cudaError_t e = bf16 ? launch(moe_compact_kernel<__nv_bfloat16>, dim3(M.L1.nchunks, E), dim3(CH), 0, st, pdl, a)
                         : launch(moe_compact_kernel<__half>, dim3(M.L1.nchunks, E), dim3(CH), 0, st, pdl, a);
    if (e != cudaSuccess) return cuda_status(e);
    e = bf16 ? launch_moe_gemv<true, 1>(a, M.L1.tiles, M.L1.S, st) : launch_moe_gemv<false, 1>(a, M.L1.tiles, M.L1.S, st);
    if (e != cudaSuccess) return cuda_status(e);
    e = bf16 ? launch_moe_gemv<true, 2>(a, M.L2.tiles, M.L2.S, st) : launch_moe_gemv<false, 2>(a, M.L2.tiles, M.L2.S, st);
    if (e != cudaSuccess) return cuda_status(e);
    e = launch(moe_combine_kernel, dim3((D + 255) / 256, B), dim3(256), 0, st, pdl, a);
    return cuda_status(e);
}

}  // extern "C"
