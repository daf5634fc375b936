// Kernels of the decode-time sparse FC (Eq. 2-3, Eq. 6, Alg. 3): chunk-local compaction and the
// split-K gather-GEMV with a fixed-order second-pass reduction.  Internal header shared by the
// FC, SwiGLU and MoE entry points.
#pragma once

#include "scap_common.cuh"

namespace scap {

enum { MODE_GATHER = 0, MODE_DENSE = 1 };
enum { EPI_BIAS = 0, EPI_GLU = 1 };

// ------------------------------------------------------------------------------------------------
// Compaction of one chunk of CH channels by a 256-thread CTA.  Thread t owns channel `k`; `keepmask`
// bit b says row b keeps it (|d[b]| >= tau).  Channels kept by any row are written in ascending
// order to idx_local[chunk*CH + j], their per-row pruned values (d where kept, else 0) to
// xs_local[b*Kpad + chunk*CH + j], and the chunk's count to counts[chunk].  Consumers turn the
// per-chunk counts into global ranks themselves, so no cross-CTA prefix sum or wait is needed.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void compact_chunk(uint32_t k, const float (&d)[SCAP_MAX_BATCH], uint32_t keepmask, int B,
                                              int chunk, int *__restrict__ counts, uint32_t *__restrict__ idx_local,
                                              float *__restrict__ xs_local, int Kpad, int *s_wcount) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool any = keepmask != 0;
    const unsigned bal = __ballot_sync(0xffffffffu, any);
    const int pre = __popc(bal & ((1u << lane) - 1u));
    if (lane == 0) s_wcount[warp] = __popc(bal);
    __syncthreads();
    int woff = 0, total = 0;
#pragma unroll
    for (int w = 0; w < CH / 32; ++w) {
        const int c = s_wcount[w];
        if (w < warp) woff += c;
        total += c;
    }
    if (any) {
        const size_t pos = (size_t)chunk * CH + woff + pre;
        idx_local[pos] = k;
#pragma unroll
        for (int b = 0; b < SCAP_MAX_BATCH; ++b)
            if (b < B) xs_local[(size_t)b * Kpad + pos] = ((keepmask >> b) & 1u) ? d[b] : 0.0f;
    }
    if (threadIdx.x == 0) counts[chunk] = total;
}

// Centre + threshold of one channel for every batch row (Alg. 3): one binary32 subtraction, one compare.
// Row b of the batch is row in_rows[b] of x (in_rows == NULL: row b).
template <typename XT>
__device__ __forceinline__ uint32_t centre_threshold(const XT *__restrict__ x, size_t row_stride, const int *in_rows,
                                                     const float *__restrict__ m, float tau, int B, int k,
                                                     float (&d)[SCAP_MAX_BATCH]) {
    uint32_t keepmask = 0;
    const float mk = m ? __ldg(m + k) : 0.0f;
#pragma unroll
    for (int b = 0; b < SCAP_MAX_BATCH; ++b) {
        d[b] = 0.0f;
        if (b < B) {
            const int row = in_rows ? in_rows[b] : b;
            const float xv = widen1(x[(size_t)row * row_stride + k]);
            const float dv = m ? __fsub_rn(xv, mk) : xv;
            d[b] = dv;
            if (fabsf(dv) >= tau) keepmask |= 1u << b;
        }
    }
    return keepmask;
}

// One CTA per chunk of CH channels.  Also clears the reduction tickets of the GEMV that follows.
template <typename XT>
__global__ void __launch_bounds__(CH) compact_kernel(const XT *__restrict__ x, const float *__restrict__ m,
                                                     const float *__restrict__ tau_p, int B, int K, int *__restrict__ counts,
                                                     uint32_t *__restrict__ idx_local, float *__restrict__ xs_local, int Kpad,
                                                     int *__restrict__ tickets, int ntickets) {
    __shared__ int s_wcount[CH / 32];
    griddep_wait();               // the previous user of this workspace has finished
    griddep_launch_dependents();  // the GEMV may start launching; it waits for this grid before reading
    const int gtid = blockIdx.x * CH + threadIdx.x;
    for (int i = gtid; i < ntickets; i += gridDim.x * CH) tickets[i] = 0;
    const float tau = __ldg(tau_p);
    float d[SCAP_MAX_BATCH];
    uint32_t keepmask = 0;
    if (gtid < K) keepmask = centre_threshold<XT>(x, (size_t)K, nullptr, m, tau, B, gtid, d);
    compact_chunk((uint32_t)gtid, d, keepmask, B, blockIdx.x, counts, idx_local, xs_local, Kpad, s_wcount);
}

// ------------------------------------------------------------------------------------------------
// Gather-GEMV arguments.  Columns are organised as `halves` groups of Nh columns (1 x N for a plain
// FC; 2 x F for the packed gate|up weight), each cut into tiles of TN columns.
// ------------------------------------------------------------------------------------------------
struct GemvArgs {
    const void *W;   // [K, ldw] storage dtype
    int K, ldw;      // ldw = total columns of a weight row
    int halves, Nh;  // column groups and columns per group (halves * Nh == ldw)
    int B, S;
    // MODE_GATHER: chunk-local lists written by the compaction
    const int *counts;
    const uint32_t *idx_local;
    const float *xs_local;
    int Kpad, nchunks;
    // MODE_DENSE: the activation itself, [B, K]
    const void *x;
    // second pass
    float *partials;  // [S, B, ldw]
    int *tickets;     // one per tile (EPI_BIAS) or per tile pair (EPI_GLU)
    // EPI_BIAS
    const float *bias;    // fp32 [ldw] or NULL
    const void *bias16;   // storage-dtype bias added on top (bias folding), or NULL
    float *y;             // row b of the result goes to y + out_rows[b] * ldw  (out_rows == NULL: row b)
    const int *out_rows;
    uint32_t *idx_out;    // optional: global ascending list of fetched channels
    int *nnz_out;         // optional
    // EPI_GLU: z = up * silu(gate), then the compaction of z for the down projection
    const float *m2, *tau2;
    float *z_out;  // optional [B, Nh]
    int *counts2;
    uint32_t *idx_local2;
    float *xs_local2;
    int Kpad2;
    int *tickets_next;  // tickets of the next GEMV, cleared here, or NULL
    int ntickets_next;
};

template <bool BF16, int BT>
__device__ __forceinline__ void fma_row(float (&acc)[BT][8], const uint4 &v, const float *__restrict__ s_xs, int i) {
    float w[8];
    widen2<BF16>(v.x, w[0], w[1]);
    widen2<BF16>(v.y, w[2], w[3]);
    widen2<BF16>(v.z, w[4], w[5]);
    widen2<BF16>(v.w, w[6], w[7]);
#pragma unroll
    for (int b = 0; b < BT; ++b) {
        const float xv = s_xs[b * LB + i];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[b][j] = fmaf(xv, w[j], acc[b][j]);
    }
}

template <bool BF16>
__device__ __forceinline__ float load_bias(const GemvArgs &a, int n) {
    float bv = a.bias ? __ldg(a.bias + n) : 0.0f;
    if (a.bias16) bv += widen_at<BF16>(a.bias16, n);
    return bv;
}

// Body of the gather-GEMV for column tile `tile` and split-K slice `s`; all 256 threads of the CTA call it.
template <bool BF16, int BT, int MODE, typename XT, int EPI>
__device__ __forceinline__ void gemv_body(const GemvArgs &a, const int tile, const int s) {
    constexpr int RB = BT < 4 ? BT : 4;  // batch rows reduced across warps per round
    constexpr int U = BT <= 2 ? 8 : 4;   // weight rows in flight per thread
    constexpr int STAGE_BYTES = LB * 4 * (1 + BT);
    constexpr int RED_BYTES = GEMV_WARPS * RB * TN * 4;
    constexpr int MAIN_BYTES = STAGE_BYTES > RED_BYTES ? STAGE_BYTES : RED_BYTES;
    __shared__ __align__(16) unsigned char s_main[MAIN_BYTES];
    __shared__ int s_prefix[MODE == MODE_GATHER ? MAX_CHUNKS_SMEM + 1 : 1];
    __shared__ int s_wcount[GEMV_WARPS];
    __shared__ int s_last;
    uint32_t *s_k = reinterpret_cast<uint32_t *>(s_main);
    float *s_xs = reinterpret_cast<float *>(s_main) + LB;
    float *s_red = reinterpret_cast<float *>(s_main);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tiles_h = (a.Nh + TN - 1) / TN;
    const int half = tile / tiles_h, tl = tile - half * tiles_h;
    const int n0 = half * a.Nh + tl * TN;  // first column of this tile
    const int n_lim = half * a.Nh + a.Nh;  // end of this column group
    const int col = n0 + lane * 8;         // this thread's 8 columns
    const bool col_ok = col < n_lim;       // Nh is a multiple of 8: all 8 or none
    const int B = a.B;

    int nnz;
    if constexpr (MODE == MODE_GATHER) {
        // global ranks from the per-chunk counts: inclusive scan by warp 0, 32 chunks at a time
        if (warp == 0) {
            int carry = 0;
            if (lane == 0) s_prefix[0] = 0;
            for (int c0 = 0; c0 < a.nchunks; c0 += 32) {
                int v = (c0 + lane < a.nchunks) ? __ldcg(a.counts + c0 + lane) : 0;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int t = __shfl_up_sync(0xffffffffu, v, o);
                    if (lane >= o) v += t;
                }
                if (c0 + lane < a.nchunks) s_prefix[c0 + lane + 1] = carry + v;
                carry += __shfl_sync(0xffffffffu, v, 31);
            }
        }
        __syncthreads();
        nnz = s_prefix[a.nchunks];
        if (EPI == EPI_BIAS && a.nnz_out && tile == 0 && s == 0 && tid == 0) *a.nnz_out = nnz;
    } else {
        nnz = a.K;
    }
    const int r0 = (int)(((long long)nnz * s) / a.S);
    const int r1 = (int)(((long long)nnz * (s + 1)) / a.S);

    float acc[BT][8];
#pragma unroll
    for (int b = 0; b < BT; ++b)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[b][j] = 0.0f;

    const unsigned char *Wb = reinterpret_cast<const unsigned char *>(a.W) + (size_t)col * 2;
    const size_t row_bytes = (size_t)a.ldw * 2;

    for (int base = r0; base < r1; base += LB) {
        const int cnt = min(LB, r1 - base);
        // ---- stage this sub-slice's channel indices and pruned activations
        if (tid < cnt) {
            const int r = base + tid;
            if constexpr (MODE == MODE_GATHER) {
                int lo = 0, hi = a.nchunks;  // find chunk c with prefix[c] <= r < prefix[c+1]
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (s_prefix[mid] <= r) lo = mid; else hi = mid;
                }
                const size_t pos = (size_t)lo * CH + (r - s_prefix[lo]);
                const uint32_t k = __ldcg(a.idx_local + pos);
                s_k[tid] = k;
#pragma unroll
                for (int b = 0; b < BT; ++b)
                    s_xs[b * LB + tid] = (b < B) ? __ldcg(a.xs_local + (size_t)b * a.Kpad + pos) : 0.0f;
                if (EPI == EPI_BIAS && a.idx_out && tile == 0) a.idx_out[r] = k;
            } else {
                s_k[tid] = (uint32_t)r;
                const XT *xp = reinterpret_cast<const XT *>(a.x);
#pragma unroll
                for (int b = 0; b < BT; ++b) s_xs[b * LB + tid] = (b < B) ? widen1(xp[(size_t)b * a.K + r]) : 0.0f;
            }
        }
        __syncthreads();
        // ---- stream the rows: warp w takes rows w, w+8, ...; U independent 16-byte loads in flight per thread
        if (col_ok) {
            for (int i0 = warp; i0 < cnt; i0 += GEMV_WARPS * U) {
                uint4 buf[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int i = i0 + GEMV_WARPS * u;
                    if (i < cnt) buf[u] = ld_stream16(Wb + (size_t)s_k[i] * row_bytes);
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int i = i0 + GEMV_WARPS * u;
                    if (i < cnt) fma_row<BF16, BT>(acc, buf[u], s_xs, i);
                }
            }
        }
        __syncthreads();
    }

    // ---- cross-warp reduction in a fixed order; thread t then owns column n0 + t
    const int ncol = n0 + tid;
    const bool ncol_ok = ncol < n_lim;
    const bool direct = (EPI == EPI_BIAS) && a.S == 1;
#pragma unroll
    for (int b0 = 0; b0 < BT; b0 += RB) {
#pragma unroll
        for (int rb = 0; rb < RB; ++rb) {
            float4 *dst = reinterpret_cast<float4 *>(s_red + ((warp * RB + rb) * TN + lane * 8));
            dst[0] = make_float4(acc[b0 + rb][0], acc[b0 + rb][1], acc[b0 + rb][2], acc[b0 + rb][3]);
            dst[1] = make_float4(acc[b0 + rb][4], acc[b0 + rb][5], acc[b0 + rb][6], acc[b0 + rb][7]);
        }
        __syncthreads();
#pragma unroll
        for (int rb = 0; rb < RB; ++rb) {
            const int b = b0 + rb;
            if (b < B && ncol_ok) {
                float v = 0.0f;
#pragma unroll
                for (int w = 0; w < GEMV_WARPS; ++w) v += s_red[(w * RB + rb) * TN + tid];
                if (direct) {
                    const int row = a.out_rows ? a.out_rows[b] : b;
                    a.y[(size_t)row * a.ldw + ncol] = load_bias<BF16>(a, ncol) + v;
                } else {
                    a.partials[((size_t)s * B + b) * a.ldw + ncol] = v;
                }
            }
        }
        __syncthreads();
    }
    if (direct) return;

    // ---- second pass: the CTA that completes a tile (integer ticket only) sums the S partials in
    // slice order, so the result does not depend on which CTA arrives last.
    __threadfence();
    __syncthreads();
    const int expected = (EPI == EPI_GLU) ? 2 * a.S : a.S;
    if (tid == 0) {
        const int t = atomicAdd(a.tickets + (EPI == EPI_GLU ? tl : tile), 1);
        s_last = (t == expected - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    if constexpr (EPI == EPI_BIAS) {
        if (ncol_ok) {
            const float bv = load_bias<BF16>(a, ncol);
            for (int b = 0; b < B; ++b) {
                float v = bv;
                for (int ss = 0; ss < a.S; ++ss) v += __ldcg(a.partials + ((size_t)ss * B + b) * a.ldw + ncol);
                const int row = a.out_rows ? a.out_rows[b] : b;
                a.y[(size_t)row * a.ldw + ncol] = v;
            }
        }
    } else {
        // gate column f and up column F + f are both complete: z, then centre + threshold + compaction of
        // z for the down projection (chunk index = tile index, since CH == TN).
        const int F = a.Nh;
        const int f = tl * TN + tid;
        if (a.tickets_next)
            for (int i = tl * TN + tid; i < a.ntickets_next; i += tiles_h * TN) a.tickets_next[i] = 0;
        float d[SCAP_MAX_BATCH];
        uint32_t keepmask = 0;
#pragma unroll
        for (int b = 0; b < SCAP_MAX_BATCH; ++b) d[b] = 0.0f;
        if (f < F) {
            const float bg = a.bias ? __ldg(a.bias + f) : 0.0f;
            const float bu = a.bias ? __ldg(a.bias + F + f) : 0.0f;
            const float tau2 = __ldg(a.tau2);
            const float mk = a.m2 ? __ldg(a.m2 + f) : 0.0f;
#pragma unroll
            for (int b = 0; b < SCAP_MAX_BATCH; ++b) {
                if (b < B) {
                    float g = bg, u = bu;
                    for (int ss = 0; ss < a.S; ++ss) {
                        g += __ldcg(a.partials + ((size_t)ss * B + b) * a.ldw + f);
                        u += __ldcg(a.partials + ((size_t)ss * B + b) * a.ldw + F + f);
                    }
                    const float z = u * (g / (1.0f + expf(-g)));
                    if (a.z_out) {
                        const int row = a.out_rows ? a.out_rows[b] : b;
                        a.z_out[(size_t)row * F + f] = z;
                    }
                    const float dv = a.m2 ? __fsub_rn(z, mk) : z;
                    d[b] = dv;
                    if (fabsf(dv) >= tau2) keepmask |= 1u << b;
                }
            }
        }
        compact_chunk((uint32_t)f, d, keepmask, B, tl, a.counts2, a.idx_local2, a.xs_local2, a.Kpad2, s_wcount);
    }
}

constexpr int gemv_min_blocks(int BT) { return BT <= 2 ? 4 : BT <= 4 ? 2 : 1; }

// blockIdx.x = column tile, blockIdx.y = split-K slice.
template <bool BF16, int BT, int MODE, typename XT, int EPI>
__global__ void __launch_bounds__(GEMV_THREADS, gemv_min_blocks(BT)) gemv_kernel(const GemvArgs a) {
    griddep_wait();
    griddep_launch_dependents();
    gemv_body<BF16, BT, MODE, XT, EPI>(a, blockIdx.x, blockIdx.y);
}

// ---- host-side plumbing shared by the entry points ------------------------------------------------

int choose_split(int K, int tiles_total);

struct FcLayout {  // byte offsets into a workspace
    int nchunks, Kpad, tiles, S;
    size_t counts, tickets, idx_local, xs_local, partials, total;
};
// Layout for one FC with N = halves * Nh columns, starting at byte offset `base`.
FcLayout fc_layout(int B, int K, int N, int halves, size_t base);
// Fills the gather-side and second-pass fields of `a` from a layout.
void bind_layout(GemvArgs &a, const FcLayout &L, unsigned char *ws);

template <typename XT>
cudaError_t launch_compact(const XT *x, const float *m, const float *tau, int B, int K, const FcLayout &L, unsigned char *ws,
                           int ntickets, cudaStream_t st);
cudaError_t launch_gemv(bool bf16, int mode, int xkind /*0 f16, 1 bf16, 2 f32; dense only*/, int epi, const GemvArgs &a,
                        cudaStream_t st);

// Inspection helper: expands chunk-local kept lists into the global ascending list (one small CTA).
cudaError_t launch_expand_idx(const int *counts, const uint32_t *idx_local, int nchunks, uint32_t *idx_out, int *nnz_out,
                              cudaStream_t st);

inline int batch_tile(int B) { return B <= 1 ? 1 : B <= 2 ? 2 : B <= 4 ? 4 : B <= 8 ? 8 : 16; }

}  // namespace scap
