// Mixture-of-experts FFN layer: a one-CTA routing kernel (softmax, top-k, renormalise), the two SwiGLU
// kernels as grouped launches with blockIdx.z = expert (experts without rows exit at once), and a small
// kernel that forms the weighted sum in selection order.
#include <string.h>

#include "scap_fc.cuh"

namespace scap {

struct Route {  // device-resident routing table
    int nb[SCAP_MAX_EXPERTS];                     // rows routed to each expert
    int rows[SCAP_MAX_EXPERTS][SCAP_MAX_BATCH];   // their batch rows, ascending
    int slots[SCAP_MAX_EXPERTS][SCAP_MAX_BATCH];  // row * top_k + position in the row's selection
    float w[SCAP_MAX_BATCH][SCAP_MAX_TOP_K];      // renormalised weights, selection order
};

struct MoeArgs {
    scap_expert ex[SCAP_MAX_EXPERTS];
    int E, top_k, B, D, F, S1, S2, tn1, tn2;
    int l2_hints;  // as FcArgs::l2_hints, for the FMA bodies
    const void *h;
    const float *logits;
    unsigned char *groups;  // per-expert scratch: z[B, F]
    size_t group_bytes;
    Route *route;
    float *yslot;  // [B * top_k, D]
    float *y;
    int *expert_out;
    float *weight_out;
};

// Selection compares the logits themselves (softmax is monotonic), ties to the lower index; the
// renormalised weights exp(l_j - max) / sum over the selected are computed in binary64.
__global__ void __launch_bounds__(64) moe_route_kernel(const float *__restrict__ logits, int B, int E, int top_k,
                                                       Route *__restrict__ r, int *__restrict__ expert_out,
                                                       float *__restrict__ weight_out) {
    __shared__ int s_sel[SCAP_MAX_BATCH * SCAP_MAX_TOP_K];
    griddep_wait();
    griddep_launch_dependents();
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
            s_sel[tid * SCAP_MAX_TOP_K + j] = best;
            p[j] = exp((double)lg[best] - (double)mx);
            tot += p[j];
        }
        for (int j = 0; j < top_k; ++j) {
            const float wv = (float)(p[j] / tot);
            r->w[tid][j] = wv;
            if (expert_out) expert_out[tid * top_k + j] = s_sel[tid * SCAP_MAX_TOP_K + j];
            if (weight_out) weight_out[tid * top_k + j] = wv;
        }
    }
    __syncthreads();
    if (tid < E) {
        int n = 0;
        for (int b = 0; b < B; ++b)
            for (int j = 0; j < top_k; ++j)
                if (s_sel[b * SCAP_MAX_TOP_K + j] == tid) {
                    r->rows[tid][n] = b;
                    r->slots[tid][n] = b * top_k + j;
                    ++n;
                }
        r->nb[tid] = n;
    }
}

// grid (tiles, S, E).  STAGE 1: packed gate|up FC of the rows routed to expert blockIdx.z, writing that
// expert's z; STAGE 2: down FC reading z and writing each row to its (row, selection position) slot.
template <bool BF16, int BT, int STAGE, int TNT>
__global__ void __launch_bounds__(FC_THREADS, fc_min_blocks(BT)) moe_fc_kernel(const MoeArgs a) {
    using ST = typename std::conditional<BF16, __nv_bfloat16, __half>::type;
    static_assert(fc_smem_for(BT) >= fc_smem_bytes(BT <= 4 ? BT : 4), "the FMA bodies for small experts use the kernel's shared memory");
    griddep_wait();
    griddep_launch_dependents();
    const int e = blockIdx.z;
    __shared__ int s_nb;  // one L2 read per CTA (written by the routing kernel just before), then broadcast
    if (threadIdx.x == 0) s_nb = __ldcg(&a.route->nb[e]);
    __syncthreads();
    const int nb = s_nb;
    if (nb == 0) return;  // the whole cluster belongs to this expert, so every CTA of it leaves together
    float *z = reinterpret_cast<float *>(a.groups + (size_t)e * a.group_bytes);
    FcArgs g = {};
    g.B = nb;
    g.l2_hints = a.l2_hints;
    if constexpr (STAGE == 1) {
        g.W = a.ex[e].Wgu; g.K = a.D; g.ldw = 2 * a.F; g.Nh = a.F; g.S = a.S1;
        g.x = a.h; g.x_ld = a.D; g.in_rows = a.route->rows[e];
        g.m = a.ex[e].m1; g.tau = a.ex[e].tau1; g.bias = a.ex[e].bgu_fused;
        g.y = z; g.y_ld = a.F;
        // an expert that got up to four rows of a larger batch takes the FMA body (cluster-uniform choice)
        if constexpr (is_mma(BT)) {
            if (nb <= 2) fc_body<BF16, 2, MODE_GATHER, ST, EPI_GLU, TNT>(g, blockIdx.x, blockIdx.y, false);
            else if (nb <= 4) fc_body<BF16, 4, MODE_GATHER, ST, EPI_GLU, TNT>(g, blockIdx.x, blockIdx.y, false);
            else fc_body_mma<BF16, BT, MODE_GATHER, ST, EPI_GLU, TNT>(g, blockIdx.x, blockIdx.y, false);
        } else {
            fc_body<BF16, BT, MODE_GATHER, ST, EPI_GLU, TNT>(g, blockIdx.x, blockIdx.y, false);
        }
    } else {
        g.W = a.ex[e].Wd; g.K = a.F; g.ldw = a.D; g.Nh = a.D; g.S = a.S2;
        g.x = z; g.x_ld = a.F;
        g.m = a.ex[e].m2; g.tau = a.ex[e].tau2; g.bias = a.ex[e].bd_fused;
        g.y = a.yslot; g.y_ld = a.D; g.out_rows = a.route->slots[e];
        if constexpr (is_mma(BT)) {
            if (nb <= 2) fc_body<BF16, 2, MODE_GATHER, float, EPI_BIAS, TNT>(g, blockIdx.x, blockIdx.y, false);
            else if (nb <= 4) fc_body<BF16, 4, MODE_GATHER, float, EPI_BIAS, TNT>(g, blockIdx.x, blockIdx.y, false);
            else fc_body_mma<BF16, BT, MODE_GATHER, float, EPI_BIAS, TNT>(g, blockIdx.x, blockIdx.y, false);
        } else {
            fc_body<BF16, BT, MODE_GATHER, float, EPI_BIAS, TNT>(g, blockIdx.x, blockIdx.y, false);
        }
    }
}

// y[b, n] = sum_j w[b, j] * yslot[b * top_k + j, n], j ascending (selection order).
__global__ void __launch_bounds__(256) moe_combine_kernel(const Route *__restrict__ r, const float *__restrict__ yslot,
                                                          float *__restrict__ y, int D, int top_k) {
    griddep_wait();
    griddep_launch_dependents();
    const int n = blockIdx.x * blockDim.x + threadIdx.x, b = blockIdx.y;
    if (n >= D) return;
    float acc = 0.0f;
    for (int j = 0; j < top_k; ++j) acc = fmaf(__ldcg(&r->w[b][j]), __ldcg(yslot + (size_t)(b * top_k + j) * D + n), acc);
    y[(size_t)b * D + n] = acc;
}

struct MoeLayout {
    size_t route, groups, group_bytes, yslot, total;
};

static MoeLayout moe_layout(int B, int D, int F, int E, int top_k) {
    MoeLayout M;
    M.route = 0;
    M.groups = align_up(sizeof(Route), 256);
    M.group_bytes = align_up(sizeof(float) * (size_t)B * F, 256);
    M.yslot = M.groups + M.group_bytes * E;
    M.total = M.yslot + align_up(sizeof(float) * (size_t)B * top_k * D, 256);
    return M;
}

template <bool BF16, int BT, int STAGE, int TNT>
static cudaError_t launch_moe_fc_tn(const MoeArgs &a, int tiles, int S, cudaStream_t st) {
    static SmemOptIn opt_in;
    auto kern = moe_fc_kernel<BF16, BT, STAGE, TNT>;
    cudaError_t e0 = ensure_dynamic_smem(kern, fc_smem_for(BT), opt_in);
    if (e0 != cudaSuccess) return e0;
    return launch_cluster(kern, dim3(tiles, S, a.E), dim3(FC_THREADS), fc_smem_for(BT), S, st, g_tune.pdl != 0, a);
}

template <bool BF16, int BT, int STAGE>
static cudaError_t launch_moe_fc_t(const MoeArgs &a, int tiles, int S, cudaStream_t st) {
    const int tn = STAGE == 1 ? a.tn1 : a.tn2;
    return tn == 128 ? launch_moe_fc_tn<BF16, BT, STAGE, 128>(a, tiles, S, st) : launch_moe_fc_tn<BF16, BT, STAGE, 256>(a, tiles, S, st);
}

template <bool BF16, int STAGE>
static cudaError_t launch_moe_fc(const MoeArgs &a, int tiles, int S, cudaStream_t st) {
    switch (batch_tile(a.B)) {
        case 1: return launch_moe_fc_t<BF16, 1, STAGE>(a, tiles, S, st);
        case 2: return launch_moe_fc_t<BF16, 2, STAGE>(a, tiles, S, st);
        case 8: return launch_moe_fc_t<BF16, 8, STAGE>(a, tiles, S, st);
        default: return launch_moe_fc_t<BF16, 16, STAGE>(a, tiles, S, st);
    }
}

}  // namespace scap

using namespace scap;

extern "C" {

size_t scap_moe_workspace(int B, int D, int F, int E, int top_k) {
    if (B < 1 || B > SCAP_MAX_BATCH || D < 1 || F < 1 || D > SCAP_MAX_K || F > SCAP_MAX_K || E < 1 || E > SCAP_MAX_EXPERTS ||
        top_k < 1 || top_k > SCAP_MAX_TOP_K || top_k > E)
        return 0;
    return moe_layout(B, D, F, E, top_k).total;
}

scap_status scap_moe_ffn(const void *h, const float *logits, const scap_expert *experts_host, int E, int top_k, float *y, int B,
                         int D, int F, scap_dtype dt, int *expert_out, float *weight_out, void *ws, size_t ws_bytes,
                         scap_stream_t stream) {
    if (!h || !logits || !experts_host || !y || !ws) return SCAP_ERR_INVALID_ARG;
    if (dt != SCAP_F16 && dt != SCAP_BF16) return SCAP_ERR_DTYPE;
    if (B < 1 || B > SCAP_MAX_BATCH || D < 1 || F < 1 || D > SCAP_MAX_K || F > SCAP_MAX_K || E < 1 || E > SCAP_MAX_EXPERTS ||
        top_k < 1 || top_k > SCAP_MAX_TOP_K || top_k > E)
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
    unsigned char *w = static_cast<unsigned char *>(ws);
    MoeArgs a;
    memset(&a, 0, sizeof(a));
    memcpy(a.ex, experts_host, sizeof(scap_expert) * E);
    a.E = E; a.top_k = top_k; a.B = B; a.D = D; a.F = F;
    a.l2_hints = g_tune.l2_hints;
    a.h = h; a.logits = logits;
    a.groups = w + M.groups;
    a.group_bytes = M.group_bytes;
    a.route = reinterpret_cast<Route *>(w + M.route);
    a.yslot = reinterpret_cast<float *>(w + M.yslot);
    a.y = y; a.expert_out = expert_out; a.weight_out = weight_out;
    const int active = B * top_k < E ? B * top_k : E;  // experts that can have rows at once
    choose_config(D, F, EPI_GLU, active, B, &a.tn1, &a.S1);
    choose_config(F, D, EPI_BIAS, active, B, &a.tn2, &a.S2);
    const int tiles1 = fc_tiles(F, EPI_GLU, a.tn1), tiles2 = fc_tiles(D, EPI_BIAS, a.tn2);
    const bool bf16 = dt == SCAP_BF16, pdl = g_tune.pdl != 0;

    cudaError_t e = launch(moe_route_kernel, dim3(1), dim3(64), 0, st, pdl, logits, B, E, top_k, a.route, expert_out, weight_out);
    if (e != cudaSuccess) return cuda_status(e);
    e = bf16 ? launch_moe_fc<true, 1>(a, tiles1, a.S1, st) : launch_moe_fc<false, 1>(a, tiles1, a.S1, st);
    if (e != cudaSuccess) return cuda_status(e);
    e = bf16 ? launch_moe_fc<true, 2>(a, tiles2, a.S2, st) : launch_moe_fc<false, 2>(a, tiles2, a.S2, st);
    if (e != cudaSuccess) return cuda_status(e);
    e = launch(moe_combine_kernel, dim3((D + 255) / 256, B), dim3(256), 0, st, pdl, (const Route *)a.route,
               (const float *)a.yslot, y, D, top_k);
    return cuda_status(e);
}

}  // extern "C"
