// Sparse FC over a batch whose rows come in groups with their own union masks (Appendix C of the paper: the union mask
// of a batch loses its sparsity when the rows' patterns do not overlap; rows that do share a pattern - the beams of
// one prompt, the tokens of one request - keep it).  The caller names the group of every row; each group is one
// z-slice of the grid and runs the ordinary FC body on its own rows (read and written through a row map), so a group
// fetches only the weight rows its own rows keep.  Up to 64 rows in up to 16 groups of at most 16 rows.
#include <string.h>

#include "scap_fc.cuh"

namespace scap {

constexpr int GR_MAX_ROWS = 64;
constexpr int GR_MAX_GROUPS = 16;

struct GroupTable {  // passed by value
    int nb[GR_MAX_GROUPS];                              // rows of each group
    unsigned char rows[GR_MAX_GROUPS][SCAP_MAX_BATCH];  // their row numbers, ascending
};

struct GroupedArgs {
    FcArgs f;
    int nb[GR_MAX_GROUPS];
    const int *rows_dev;  // [GR_MAX_GROUPS][SCAP_MAX_BATCH], written by group_table_kernel
};

// The row maps have to be in device memory (the FC body reads them through a pointer): one tiny kernel copies them out
// of its parameters.
__global__ void __launch_bounds__(256) group_table_kernel(const GroupTable t, int *__restrict__ rows_dev) {
    griddep_wait();               // the previous kernel in the stream may still read the table
    griddep_launch_dependents();
    const int i = threadIdx.x;
    if (i < GR_MAX_GROUPS * SCAP_MAX_BATCH) rows_dev[i] = t.rows[i / SCAP_MAX_BATCH][i % SCAP_MAX_BATCH];
}

// grid (tiles, S, groups).  BT: 2 (groups of one or two rows, fp32 FMA) or 8 / 16 (tensor-core body; a group of up to
// four rows inside such a launch takes the FMA body, a cluster-uniform choice).
template <bool BF16, int BT, int TNT>
__global__ void __launch_bounds__(FC_THREADS, fc_min_blocks(BT)) grouped_fc_kernel(const GroupedArgs a) {
    using ST = typename std::conditional<BF16, __nv_bfloat16, __half>::type;
    griddep_wait();
    griddep_launch_dependents();
    const int g = blockIdx.z, nb = a.nb[g];
    if (nb == 0) return;  // the whole cluster belongs to this group
    FcArgs f = a.f;
    f.B = nb;
    f.in_rows = a.rows_dev + g * SCAP_MAX_BATCH;
    f.out_rows = f.in_rows;
    if constexpr (is_mma(BT)) {
        if (nb <= 2) fc_body<BF16, 2, MODE_GATHER, ST, EPI_BIAS, TNT>(f, blockIdx.x, blockIdx.y, false);
        else if (nb <= 4) fc_body<BF16, 4, MODE_GATHER, ST, EPI_BIAS, TNT>(f, blockIdx.x, blockIdx.y, false);
        else fc_body_mma<BF16, BT, MODE_GATHER, ST, EPI_BIAS, TNT>(f, blockIdx.x, blockIdx.y, false);
    } else {
        fc_body<BF16, BT, MODE_GATHER, ST, EPI_BIAS, TNT>(f, blockIdx.x, blockIdx.y, false);
    }
}

template <bool BF16, int BT, int TNT>
static cudaError_t launch_grouped_tn(const GroupedArgs &a, int tiles, int groups, cudaStream_t st) {
    static SmemOptIn opt_in;
    auto kern = grouped_fc_kernel<BF16, BT, TNT>;
    constexpr int smem = is_mma(BT) ? (fc_smem_for(BT) > fc_smem_bytes(4) ? fc_smem_for(BT) : fc_smem_bytes(4)) : fc_smem_bytes(BT);
    cudaError_t e0 = ensure_dynamic_smem(kern, smem, opt_in);
    if (e0 != cudaSuccess) return e0;
    return launch_cluster(kern, dim3(tiles, a.f.S, groups), dim3(FC_THREADS), smem, a.f.S, st, g_tune.pdl != 0, a);
}

template <bool BF16, int BT>
static cudaError_t launch_grouped_t(const GroupedArgs &a, int tiles, int groups, cudaStream_t st) {
    return a.f.tn == 128 ? launch_grouped_tn<BF16, BT, 128>(a, tiles, groups, st) : launch_grouped_tn<BF16, BT, 256>(a, tiles, groups, st);
}

template <bool BF16>
static cudaError_t launch_grouped(const GroupedArgs &a, int max_nb, int tiles, int groups, cudaStream_t st) {
    if (max_nb <= 2) return launch_grouped_t<BF16, 2>(a, tiles, groups, st);
    if (max_nb <= 8) return launch_grouped_t<BF16, 8>(a, tiles, groups, st);
    return launch_grouped_t<BF16, 16>(a, tiles, groups, st);
}

}  // namespace scap

using namespace scap;

extern "C" {

size_t scap_grouped_workspace(void) { return align_up(sizeof(int) * GR_MAX_GROUPS * SCAP_MAX_BATCH, 256); }

scap_status scap_sparse_fc_grouped(const void *x, const void *W, const float *m, const float *tau, const float *b_fused, float *y,
                                   int B, int K, int N, scap_dtype dt, const int *group_of_row_host, void *ws, size_t ws_bytes,
                                   scap_stream_t stream) {
    if (!x || !W || !tau || !y || !group_of_row_host || !ws) return SCAP_ERR_INVALID_ARG;
    if (dt != SCAP_F16 && dt != SCAP_BF16) return SCAP_ERR_DTYPE;
    if (B < 1 || B > GR_MAX_ROWS || K < 1 || N < 1 || K > SCAP_MAX_K) return SCAP_ERR_SHAPE;
    if (N % 8 != 0 || !aligned16(x) || !aligned16(W) || !aligned16(y) || !aligned16(ws) || (m && !aligned16(m)) ||
        (b_fused && !aligned16(b_fused)))
        return SCAP_ERR_ALIGN;
    if (ws_bytes < scap_grouped_workspace()) return SCAP_ERR_WORKSPACE;
    GroupTable t;
    memset(&t, 0, sizeof(t));
    int groups = 0, max_nb = 0, active = 0;
    for (int b = 0; b < B; ++b) {
        const int g = group_of_row_host[b];
        if (g < 0 || g >= GR_MAX_GROUPS) return SCAP_ERR_INVALID_ARG;
        if (t.nb[g] >= SCAP_MAX_BATCH) return SCAP_ERR_SHAPE;  // at most 16 rows share a mask
        t.rows[g][t.nb[g]++] = (unsigned char)b;
        if (g + 1 > groups) groups = g + 1;
    }
    for (int g = 0; g < groups; ++g) {
        if (t.nb[g] > max_nb) max_nb = t.nb[g];
        active += t.nb[g] > 0;
    }
    scap_status stt = check_device();
    if (stt != SCAP_OK) return stt;

    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    GroupedArgs a;
    memset(&a, 0, sizeof(a));
    a.f.W = W; a.f.K = K; a.f.ldw = N; a.f.Nh = N;
    choose_config(K, N, EPI_BIAS, active, max_nb, &a.f.tn, &a.f.S);
    a.f.x = x; a.f.x_ld = K; a.f.m = m; a.f.tau = tau; a.f.bias = b_fused; a.f.y = y; a.f.y_ld = N;
    a.f.l2_hints = g_tune.l2_hints;
    memcpy(a.nb, t.nb, sizeof(a.nb));
    int *rows_dev = static_cast<int *>(ws);
    a.rows_dev = rows_dev;
    cudaError_t e = launch(group_table_kernel, dim3(1), dim3(256), 0, st, g_tune.pdl != 0, t, rows_dev);
    if (e != cudaSuccess) return cuda_status(e);
    const int tiles = fc_tiles(N, EPI_BIAS, a.f.tn);
    e = dt == SCAP_BF16 ? launch_grouped<true>(a, max_nb, tiles, groups, st) : launch_grouped<false>(a, max_nb, tiles, groups, st);
    return cuda_status(e);
}

}  // extern "C"
