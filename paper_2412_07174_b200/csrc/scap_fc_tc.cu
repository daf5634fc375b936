// Batch 3..16 on the 5th-generation tensor cores: the sparse FC of Eq. 2-3 / Eq. 6 / Alg. 3 as
//   16-byte asynchronous row copies  ->  swizzled shared-memory ring  ->  tcgen05.mma  ->  accumulator in TMEM.
//
// Same decomposition as the FMA kernel (grid = 128-column tiles x S, the S CTAs of a tile form a cluster and split
// the input channels by interleaved 32-channel chunks, cluster exchange of the partial tiles at the end, two CTAs
// per SM):
//   prologue   all 8 warps: d = x - m, |d| >= tau, union over the batch, ballot compaction (ascending kept list),
//              and the pruned values split exactly into parts of the weight dtype (bf16: hi+mid+lo, fp16: hi+lo)
//              written as the A operand: row (part * B + b), K-major core matrices of 8 rows x 16 bytes;
//   7 warps    producers: a warp moves two kept rows (256 bytes of the tile each) per instruction with 16-byte
//              asynchronous copies (cp.async) straight into the rows' places in a ring stage of 64 rows = four
//              4 KB blocks, each laid out as the MN-major, 128-byte-swizzled B operand (N = 128 columns of W,
//              K = 16 rows); an asynchronous arrival per lane and stage fires when the copies have landed, so
//              producers never wait for data and the whole ring is the in-flight buffer;
//   warp 1     one lane waits per stage and issues tcgen05.mma M=128 N=128 K=16 per block of 16 rows (all parts
//              of all batch rows at once; rows of M beyond parts * B read whatever follows in shared memory and
//              produce accumulator rows nobody reads) and commits to the stage's "empty" barrier; the accumulator
//              (128 lanes x 128 fp32 columns) stays in TMEM across blocks and fills;
//   epilogue   warps 0-1 read the accumulator rows, the parts are added smallest first, and the cluster exchange
//              and bias / SwiGLU epilogue are those of the other variants.
// (A TMA row gather - cp.async.bulk.tensor tile::gather4, four rows x 128 bytes per instruction - was measured
// first and was no faster on this access pattern.)
// Every wait on an mbarrier is bounded; a wait that runs out sets a device status word, the CTA stops issuing work,
// still passes every cluster barrier and frees its TMEM.
#include <cuda.h>
#include <string.h>

#include <atomic>

#include "scap_fc.cuh"

namespace scap {

constexpr int TC_TN = 128;                          // columns per CTA
constexpr int TC_KB = 16 * TC_TN * 2;               // bytes of one block of 16 kept rows (one MMA): 4 KB
constexpr int TC_SROWS = 64;                        // kept rows per ring stage (4 blocks)
constexpr int TC_STAGE = TC_SROWS * TC_TN * 2;      // 16 KB
constexpr int TC_NST = 3;                           // ring stages (48 KB per CTA, two CTAs per SM)
constexpr int TC_CAP = 1408;                        // most kept channels per fill (44 chunks)
constexpr int TC_PLANE_DATA = TC_CAP * 32;          // A-operand bytes: 16 per channel and 8-row group, two groups at full capacity
constexpr int TC_PLANE = TC_PLANE_DATA + 2048;      // + slack for the rows of M that nobody uses
constexpr int TC_PART_LD = TC_TN + 1;               // row pitch of the accumulator copy (conflict-free)
constexpr uint32_t TC_SPIN = 1u << 20;              // polls before a wait gives up (tens of milliseconds); scap_tune("tc_spin") overrides
__host__ __device__ constexpr int tc_pu(int ROWS) { return ROWS == 8 ? 6 : 3; }  // chunks per warp per fill, at most
// 8-row groups of the A operand for B batch rows (parts stacked densely: row = part * B + b), and the chunks of 32
// channels that fit in the A-operand region with that many groups
__host__ __device__ constexpr int tc_groups(int B, int nsplit) { return (nsplit * B + 7) / 8; }
__host__ __device__ constexpr int tc_cap_chunks(int groups) {
    return TC_PLANE_DATA / (groups * 16) / 32 < TC_CAP / 32 ? TC_PLANE_DATA / (groups * 16) / 32 : TC_CAP / 32;
}

// shared-memory map (offsets from a 1024-byte aligned base)
constexpr int TC_OFF_RING = 0;
constexpr int TC_OFF_PLANE = TC_OFF_RING + TC_NST * TC_STAGE;
constexpr int TC_OFF_K = TC_OFF_PLANE + TC_PLANE;
constexpr int TC_OFF_GATHER = TC_OFF_K + TC_CAP * 4;
constexpr int TC_OFF_MISC = TC_OFF_GATHER + 16 * TC_TN * 4;
constexpr int TC_SMEM = TC_OFF_MISC + 1024 + 1024;  // misc block + alignment slack
static_assert(48 * TC_PART_LD * 4 <= TC_NST * TC_STAGE, "accumulator copy must fit in the ring");
static_assert(2 * (TC_SMEM + 1024) <= 233472, "two CTAs must fit in the shared memory of an SM");

__device__ int g_tc_status;  // 0, or the code of the first bounded wait that ran out

struct TcMisc {
    unsigned long long full[TC_NST];
    unsigned long long empty[TC_NST];
    unsigned long long fill_done;
    uint32_t tmem_base;
    int abort;
    int issued;  // the MMA lane has issued at least one MMA
    int wcnt[FC_WARPS];
    int rows[16];
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long *bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_test(unsigned long long *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false (and the status word set) when the phase did not complete within `limit` polls.
__device__ __forceinline__ bool mbar_wait(unsigned long long *bar, uint32_t parity, int code, volatile int *abort_flag,
                                          uint32_t limit) {
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_test(bar, parity)) return true;
        if (*abort_flag) return false;
        if (i > 64) __nanosleep(32);
    }
    atomicCAS(&g_tc_status, 0, code);
    *abort_flag = 1;
    return false;
}

__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void tc_commit(unsigned long long *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor (start address, leading / stride byte offsets in 16-byte units, version 1, swizzle).
__device__ __forceinline__ uint64_t tc_desc(uint32_t addr, uint32_t lbo, uint32_t sbo, uint32_t layout) {
    return (uint64_t)((addr >> 4) & 0x3fffu) | ((uint64_t)((lbo >> 4) & 0x3fffu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3fffu) << 32) | (1ull << 46) | ((uint64_t)layout << 61);
}

template <bool BF16, int ROWS, int MODE, typename XT, int EPI>
__global__ void __launch_bounds__(FC_THREADS, 2) fc_tc_kernel(const FcArgs a) {
    constexpr int TNT = TC_TN, HALF = TNT / 2, NSPLIT = mma_nsplit(BF16), PU = tc_pu(ROWS);
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char *s_ring = smem + TC_OFF_RING;
    unsigned char *s_plane = smem + TC_OFF_PLANE;
    uint32_t *s_k = reinterpret_cast<uint32_t *>(smem + TC_OFF_K);
    float *s_gather = reinterpret_cast<float *>(smem + TC_OFF_GATHER);  // this CTA's partial tile [b][TNT]
    TcMisc *misc = reinterpret_cast<TcMisc *>(smem + TC_OFF_MISC);
    float *s_part = reinterpret_cast<float *>(s_ring);                   // accumulator rows, after the stream
    volatile int *abort_flag = &misc->abort;
    const uint32_t spin = a.spin ? (uint32_t)a.spin : TC_SPIN;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tile = blockIdx.x, s = blockIdx.y;
    const int B = a.B, S = a.S, K = a.K;
    const int racc = NSPLIT * B;               // rows of the A operand (and of the accumulator) in use: part * B + b
    const int G = tc_groups(B, NSPLIT);        // 8-row groups that hold them
    const uint32_t LBO = G * 128, BLK = 2 * LBO;  // bytes: between the two K halves of a block, and per block
    const int cap_chunks = tc_cap_chunks(G);
    const XT *xg = reinterpret_cast<const XT *>(a.x);

    if (tid == 0) {
        for (int i = 0; i < TC_NST; ++i) {
            mbar_init(&misc->full[i], (FC_WARPS - 1) * 32);  // one arrival per producer lane
            mbar_init(&misc->empty[i], 1);
        }
        mbar_init(&misc->fill_done, 1);
        misc->abort = 0;
        misc->issued = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {  // the accumulator: 128 TMEM columns, allocated by warp 0 and freed by it at the end
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&misc->tmem_base)), "r"(TNT)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }

    const int per = ((EPI == EPI_GLU ? HALF : TNT) + S - 1) / S;
    float bias0[2], bias1[2];

    const int nchunks = (K + 31) >> 5;
    const int my_chunks = nchunks > s ? (nchunks - s + S - 1) / S : 0;
    float tau = 0.0f;

    griddep_wait();  // nothing (activations, row map, tau, m, biases) is read before earlier work on the stream is complete
    griddep_launch_dependents();
    if constexpr (MODE == MODE_GATHER) {
        float tv = 0.0f;
        if (lane == 0) tv = ld_act(a.tau);
        tau = __shfl_sync(0xffffffffu, tv, 0);
    }
    prefetch_bias<BF16, EPI, TNT>(a, tile, s, per, bias0, bias1);
    if (a.in_rows && tid < 16) misc->rows[tid] = __ldcg(a.in_rows + (tid < B ? tid : 0));
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = misc->tmem_base;

    uint32_t stages_done = 0;  // ring stages streamed so far by this CTA, the same in every thread
    int fills_done = 0;
    const uint32_t idesc = (1u << 4) | ((BF16 ? 1u : 0u) << 7) | ((BF16 ? 1u : 0u) << 10) | (0u << 15) | (1u << 16) |
                           ((uint32_t)(TNT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

    for (int j0 = 0; j0 < my_chunks; j0 += cap_chunks) {
        const int nj = min(cap_chunks, my_chunks - j0);
        const int pu = (nj + FC_WARPS - 1) / FC_WARPS;  // consecutive chunks per warp
        // ---- keep masks: all activation loads of a lane in flight together, values kept in registers
        float mk[PU];
        XT xraw[PU][ROWS];
        uint32_t km[PU];
        unsigned bal[PU];
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            const int j = warp * pu + p;
            const int k = (s + S * (j0 + j)) * 32 + lane;
            mk[p] = a.m ? ld_act_if(a.m + k, p < pu && j < nj && k < K) : 0.0f;
        }
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            const int j = warp * pu + p;
            const int k = (s + S * (j0 + j)) * 32 + lane;
            const bool ok = p < pu && j < nj && k < K;
#pragma unroll
            for (int b = 0; b < ROWS; ++b) {
                const int row = a.in_rows ? misc->rows[b] : b;
                xraw[p][b] = ld_act_if(xg + (size_t)row * a.x_ld + k, ok && b < B);
            }
        }
        int my_off[PU], wtotal = 0;
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            const int j = warp * pu + p;
            const int k = (s + S * (j0 + j)) * 32 + lane;
            const bool ok = p < pu && j < nj && k < K;
            uint32_t m_ = 0;
            if constexpr (MODE == MODE_GATHER) {
#pragma unroll
                for (int b = 0; b < ROWS; ++b) {
                    const float xv = widen1(xraw[p][b]);
                    const float dv = a.m ? __fsub_rn(xv, mk[p]) : xv;
                    m_ |= (ok && b < B && fabsf(dv) >= tau) ? (1u << b) : 0u;
                }
            } else {
                m_ = ok ? 1u : 0u;
            }
            km[p] = m_;
            bal[p] = __ballot_sync(0xffffffffu, m_ != 0);
            my_off[p] = wtotal;
            wtotal += __popc(bal[p]);
        }
        if (lane == 0) misc->wcnt[warp] = wtotal;
        if (MODE == MODE_GATHER && a.bits && tile == 0) {
            unsigned mine = 0;
#pragma unroll
            for (int p = 0; p < PU; ++p) mine = lane == p ? bal[p] : mine;
            const int j = warp * pu + lane;
            if (lane < pu && j < nj) a.bits[s + S * (j0 + j)] = mine;
        }
        __syncthreads();
        int cnt = 0, wbase = 0;
#pragma unroll
        for (int w = 0; w < FC_WARPS; ++w) {
            const int c = misc->wcnt[w];
            cnt += c;
            wbase += w < warp ? c : 0;
        }
        // ---- kept list and A operand.  Element (row r = part * B + b, kept position pos): block pos / 16,
        // K half (pos / 8) & 1, 8-row group r / 8, then 16 bytes per row of the group, 2 bytes per position.
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            if (km[p]) {
                const int j = warp * pu + p;
                const int k = (s + S * (j0 + j)) * 32 + lane;
                const int pos = wbase + my_off[p] + __popc(bal[p] & ((1u << lane) - 1u));
                s_k[pos] = (uint32_t)k;
                unsigned char *blk = s_plane + (size_t)(pos >> 4) * BLK + ((pos >> 3) & 1) * LBO + (pos & 7) * 2;
#pragma unroll
                for (int b = 0; b < ROWS; ++b) {
                    if (b < B) {
                        const float xv = widen1(xraw[p][b]);
                        const float dv = (MODE == MODE_GATHER && a.m) ? __fsub_rn(xv, mk[p]) : xv;
                        const bool kept = MODE == MODE_DENSE || (((km[p] >> b) & 1u) != 0);
                        unsigned short part[3];
                        split_parts<BF16>(kept ? dv : 0.0f, part);
#pragma unroll
                        for (int q = 0; q < NSPLIT; ++q) {
                            const int r = q * B + b;
                            *reinterpret_cast<unsigned short *>(blk + (r >> 3) * 128 + (r & 7) * 16) = part[q];
                        }
                    }
                }
            }
        }
        __syncthreads();
        // The last block is completed with copies of the last kept row and zero activations (a padded row adds
        // exactly 0 for finite weights).
        const int cnt_pad = (cnt + 15) & ~15;
        if (tid < 16 && cnt > 0 && cnt + tid < cnt_pad) {
            const int pos = cnt + tid;
            s_k[pos] = s_k[cnt - 1];
            unsigned char *blk = s_plane + (size_t)(pos >> 4) * BLK + ((pos >> 3) & 1) * LBO + (pos & 7) * 2;
            for (int r = 0; r < racc; ++r) *reinterpret_cast<unsigned short *>(blk + (r >> 3) * 128 + (r & 7) * 16) = 0;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the tensor core
        __syncthreads();

        const uint32_t nblk = (uint32_t)cnt_pad >> 4;
        const uint32_t nstg = ((uint32_t)cnt_pad + TC_SROWS - 1) / TC_SROWS;  // ring stages of this fill (the last may be short)
        if (warp != 1) {
            // ---- producers: stage sq of the fill holds kept rows 64 sq .. 64 sq + 63 and goes to ring slot
            // (stages_done + sq) % TC_NST; inside a stage, warp pw takes rows pw, pw + 7, ...  A row moves with one
            // 16-byte asynchronous copy per lane (global -> swizzled place in the stage, no registers in between);
            // after its rows of a stage a lane posts one asynchronous arrival on the stage's "full" barrier, which
            // fires when its copies have landed.  Producers never wait for data: the ring is the in-flight buffer.
            constexpr int P = FC_WARPS - 1;
            const int pw = warp == 0 ? 0 : warp - 1;
            const int l16 = lane & 15;  // a row of the tile is 256 bytes = 16 lanes; a warp moves two rows at once
            int col;
            if constexpr (EPI == EPI_GLU) col = (l16 >> 3) * a.Nh + tile * HALF + (l16 & 7) * 8;
            else col = tile * TNT + l16 * 8;
            const bool col_ok = EPI == EPI_GLU ? (tile * HALF + (l16 & 7) * 8 < a.Nh) : (col < a.Nh);
            const unsigned char *Wb = reinterpret_cast<const unsigned char *>(a.W) + (col_ok ? (size_t)col * 2 : 0);
            const uint32_t src_bytes = col_ok ? 16u : 0u;  // 0: the copy writes zeros
            const size_t row_bytes = (size_t)a.ldw * 2;
            const uint32_t ring = smem_u32(s_ring) + (uint32_t)(l16 >> 3) * 1024;  // + this lane's 64-column half
            for (uint32_t sq = 0; sq < nstg; ++sq) {
                const uint32_t it = stages_done + sq, st = it % TC_NST;
                bool ok = true;
                if (lane == 0) ok = mbar_wait(&misc->empty[st], ((it / TC_NST) & 1u) ^ 1u, 1, abort_flag, spin);
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                const int rows_here = min(TC_SROWS, cnt_pad - (int)sq * TC_SROWS);
                const uint32_t base = ring + st * TC_STAGE;
#pragma unroll
                for (int u = 0; u < (TC_SROWS / 2 + P - 1) / P; ++u) {
                    const int lr = 2 * (pw + P * u) + (lane >> 4);  // row inside the stage: block lr / 16, K half (lr / 8) & 1, row lr & 7
                    if (lr < rows_here) {
                        const uint32_t r = (uint32_t)lr & 7;
                        const uint32_t dst = base + ((uint32_t)lr >> 4) * TC_KB + (((uint32_t)lr >> 3) & 1) * 2048 + r * 128 + (((uint32_t)l16 & 7) ^ r) * 16;
                        const unsigned char *src = Wb + (size_t)s_k[sq * TC_SROWS + lr] * row_bytes;
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
                    }
                }
                asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(&misc->full[st])) : "memory");
            }
        } else {
            // ---- MMA issuer: one wait per stage, then one MMA per block of 16 rows in it
            for (uint32_t sq = 0; sq < nstg; ++sq) {
                const uint32_t it = stages_done + sq, st = it % TC_NST;
                bool ok = true;
                if (lane == 0) {
                    ok = mbar_wait(&misc->full[st], (it / TC_NST) & 1u, 2, abort_flag, spin);
                    if (ok) {
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // copied rows -> tensor-core proxy
                        tc_fence_after();
                        const uint32_t kb_n = min(4u, nblk - sq * 4);
                        misc->issued = 1;
                        for (uint32_t kb = 0; kb < kb_n; ++kb) {
                            const uint64_t da = tc_desc(smem_u32(s_plane) + (sq * 4 + kb) * BLK, LBO, 128, 0);
                            const uint64_t db = tc_desc(smem_u32(s_ring) + st * TC_STAGE + kb * TC_KB, 1024, 2048, 2);
                            tc_mma(tmem, da, db, idesc, (it > 0 || kb > 0) ? 1u : 0u);
                        }
                        tc_commit(&misc->empty[st]);  // arrives once the MMAs have read the stage
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
            }
            if (nblk > 0 && lane == 0 && !*abort_flag) tc_commit(&misc->fill_done);
            __syncwarp();
        }
        // ---- the A operand and the kept list are reused by the next fill: wait until this fill's MMAs are done
        if (nblk > 0) {
            if (mbar_wait(&misc->fill_done, (uint32_t)fills_done & 1u, 3, abort_flag, spin)) ++fills_done;
        }
        stages_done += nstg;
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        if (*abort_flag) break;
    }

    asm volatile("cp.async.wait_all;" ::: "memory");
    // After a wait that ran out, MMAs issued before it may still be writing the accumulator: one more commit and a wait
    // with the fixed limit (not the tunable one) let them finish before the TMEM columns are handed back.
    if (*abort_flag && misc->issued) {
        if (warp == 1 && lane == 0) tc_commit(&misc->fill_done);
        __syncwarp();
        int drain_abort = 0;
        mbar_wait(&misc->fill_done, (uint32_t)fills_done & 1u, 4, &drain_abort, TC_SPIN);
    }
    // ---- accumulator rows -> shared memory (the ring is idle now), parts added smallest first
    const bool have_acc = stages_done > 0 && !*abort_flag;
    const int acc_rows = racc;
    if (have_acc && warp * 32 < acc_rows && warp < 2) {
#pragma unroll 1
        for (int c0 = 0; c0 < TNT; c0 += 32) {
            uint32_t v[32];
            asm volatile(
                "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                  "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
                  "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
                  "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                : "r"(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0));
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            const int r = warp * 32 + lane;
            if (r < acc_rows) {
#pragma unroll
                for (int j = 0; j < 32; ++j) s_part[r * TC_PART_LD + c0 + j] = __uint_as_float(v[j]);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TNT) : "memory");
    for (int i = tid; i < 16 * TNT; i += FC_THREADS) {
        const int b = i / TNT, c = i - b * TNT;
        float v = 0.0f;
        if (have_acc && b < B) {
#pragma unroll
            for (int q = NSPLIT - 1; q >= 0; --q) v += s_part[(q * B + b) * TC_PART_LD + c];
        }
        s_gather[i] = v;
    }

    // ---- cluster exchange, pull form, and the bias / SwiGLU epilogue
    cg::cluster_group cluster = cg::this_cluster();
    if (S > 1) cluster.sync();
    else __syncthreads();
    const float *peer[MAX_CLUSTER];
#pragma unroll
    for (int q = 0; q < MAX_CLUSTER; ++q) peer[q] = (S > 1 && q < S) ? cluster.map_shared_rank(s_gather, q) : s_gather;
    for (int it = 0; tid + it * FC_THREADS < per * B; ++it) {
        const int i = tid + it * FC_THREADS;
        const int b = i / per, c = i - b * per;
        const int row = a.out_rows ? __ldcg(a.out_rows + b) : b;
        if constexpr (EPI == EPI_BIAS) {
            const int n = tile * TNT + s * per + c;
            if (s * per + c < TNT && n < a.Nh) {
                float v = it == 0 ? bias0[0] : it == 1 ? bias0[1] : load_bias<BF16>(a, n);
#pragma unroll
                for (int q = 0; q < MAX_CLUSTER; ++q)
                    if (q < S) v += peer[q][b * TNT + s * per + c];
                store_result(a, row, b, n, v);
            }
        } else {
            const int F = a.Nh, f = tile * HALF + s * per + c;
            if (s * per + c < HALF && f < F) {
                float gt = it == 0 ? bias0[0] : it == 1 ? bias0[1] : (a.bias ? __ldcg(a.bias + f) : 0.0f);
                float up = it == 0 ? bias1[0] : it == 1 ? bias1[1] : (a.bias ? __ldcg(a.bias + F + f) : 0.0f);
#pragma unroll
                for (int q = 0; q < MAX_CLUSTER; ++q)
                    if (q < S) {
                        gt += peer[q][b * TNT + s * per + c];
                        up += peer[q][b * TNT + HALF + s * per + c];
                    }
                const float z = up * (gt / (1.0f + expf(-gt)));  // up * silu(gate)
                a.y[(size_t)row * a.y_ld + f] = z;
                if (a.z_copy) a.z_copy[(size_t)b * F + f] = z;
            }
        }
    }
    if (S > 1) cluster.sync();
}

// ------------------------------------------------------------------------------------------------
// Dense-stream variant (batch 5..16).  With that many rows the union mask of independent rows keeps nearly every channel
// (Appendix C), so gathering kept rows buys nothing and costs the memory-level parallelism of the copy engine.  Here
// the CTA streams ALL rows of its share of the tile - blocks of 64 consecutive rows, block q of rank s = rows
// (q S + s) 64 .. + 63 - with two TMA box loads per block (64 columns x 64 rows each, 128-byte swizzle: exactly the
// MN-major B operand of the MMA, no address arithmetic, one instruction per 8 KB), and pruning happens on the small
// operand instead: a dropped channel gets a zero activation.  Roles: warp 0 issues the TMA loads, warp 1 the MMAs,
// warps 2-7 threshold one 32-channel chunk at a time (d = x - m, |d| >= tau, ballot for the mask words, exact split into
// parts of the weight dtype) and write it as the A operand of its stage; W ring and A ring have DS_NST stages each and
// share the stage's "empty" barrier.  The epilogue is that of the gather kernel.  Every wait is bounded.
// ------------------------------------------------------------------------------------------------
constexpr int DS_NST = 4;
constexpr int DS_STAGE_W = 64 * TC_TN * 2;                      // 16 KB: two boxes of 64 rows x 64 columns
__host__ __device__ constexpr int ds_a_stage(int groups) { return 4 * 2 * groups * 128; }  // A operand of 64 channels
constexpr int DS_OFF_W = 0;
constexpr int DS_OFF_A = DS_OFF_W + DS_NST * DS_STAGE_W;
constexpr int DS_OFF_GATHER = DS_OFF_A + DS_NST * ds_a_stage(6) + 2560;  // + slack: the MMA reads 128 rows of M, used or not
constexpr int DS_OFF_MISC = DS_OFF_GATHER + 16 * TC_TN * 4;
constexpr int DS_SMEM = DS_OFF_MISC + 512 + 1024;               // misc block + alignment slack
static_assert(48 * TC_PART_LD * 4 <= DS_NST * DS_STAGE_W, "accumulator copy must fit in the W ring");
static_assert(2 * (DS_SMEM + 1024) <= 233472, "two CTAs must fit in the shared memory of an SM");

struct DsMisc {
    unsigned long long wfull[DS_NST];   // TMA bytes of the stage have landed
    unsigned long long afull[DS_NST];   // both chunks of the stage's A operand are written
    unsigned long long empty[DS_NST];   // the stage's MMAs have read W and A
    unsigned long long done;
    unsigned long long recv;            // split-K partials of this rank's columns have landed
    uint32_t tmem_base;
    int abort;
    int issued;
    int rows[16];
};

__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// One box of the tensor map (64 columns x 64 rows) to shared memory; completion counts bytes on `bar`.  The copy goes to this CTA only.
__device__ __forceinline__ void tma_box_2d(uint32_t dst, const CUtensorMap *map, int x, int y, unsigned long long *bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
                 "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
                 : "memory");
}

template <bool BF16, int ROWS, int MODE, typename XT, int EPI>
__global__ void __launch_bounds__(FC_THREADS, 2) fc_ds_kernel(const FcArgs a, const __grid_constant__ CUtensorMap tmap) {
    constexpr int TNT = TC_TN, HALF = TNT / 2, NSPLIT = mma_nsplit(BF16);
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char *s_w = smem + DS_OFF_W;
    unsigned char *s_a = smem + DS_OFF_A;
    float *s_gather = reinterpret_cast<float *>(smem + DS_OFF_GATHER);
    DsMisc *misc = reinterpret_cast<DsMisc *>(smem + DS_OFF_MISC);
    float *s_part = reinterpret_cast<float *>(s_w);  // accumulator rows, after the stream
    volatile int *abort_flag = &misc->abort;
    const uint32_t spin = a.spin ? (uint32_t)a.spin : TC_SPIN;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tile = blockIdx.x, s = blockIdx.y;
    const int B = a.B, S = a.S, K = a.K;
    const int racc = NSPLIT * B;
    const int G = tc_groups(B, NSPLIT);
    const uint32_t LBO = G * 128, BLK = 2 * LBO, ASTG = 4 * BLK;
    const XT *xg = reinterpret_cast<const XT *>(a.x);
    const int nblk64 = (K + 63) >> 6;
    const int nq = nblk64 > s ? (nblk64 - s + S - 1) / S : 0;  // 64-row blocks (= stages) of this rank

    const int per = ((EPI == EPI_GLU ? HALF : TNT) + S - 1) / S;   // columns (gate/up pairs) a rank finishes
    const uint32_t recv_bar = smem_addr(&misc->recv);
    if (tid == 0) {
        for (int i = 0; i < DS_NST; ++i) {
            mbar_init(&misc->wfull[i], 1);
            mbar_init(&misc->afull[i], 2);
            mbar_init(&misc->empty[i], 1);
        }
        mbar_init(&misc->done, 1);
        misc->abort = 0;
        misc->issued = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (S > 1) {
            // S B (columns this rank finishes) partial sums (gate and up: twice that) will land on the receive barrier
            const int owned = max(0, min(per, (EPI == EPI_GLU ? HALF : TNT) - s * per));
            mbarrier_init(recv_bar, 1);
            mbarrier_arrive_expect(recv_bar, (uint32_t)(S * B * owned * (EPI == EPI_GLU ? 8 : 4)));
        }
    }
    // The arrival half of a cluster barrier (the fence after the initialisation publishes the receive barrier; the
    // arrival itself carries no ordering and so does not wait for anything); the waiting half sits before the first
    // send, long after every rank has arrived.
    if (S > 1) cluster_arrive_relaxed();
    // This rank's share of m and x is asked into L2 first of all, ahead of the weight stream: a request that misses L2
    // later queues behind megabytes of weight reads (measured: 1.8 - 2.8 us, which made the operand warps the limit of
    // the stream and of its start).  These are hints without a result: L2 is the point of coherence, so a line that
    // earlier work on the stream rewrites after the hint is rewritten there, and the loads proper - after the wait,
    // through L2 - see the final contents.  One line per thread and turn; every tile of the call asks for the same
    // lines, L2 merges them.
    if (warp >= 2) {
        const int t = tid - 64;
        if (MODE == MODE_GATHER && a.m) {
            for (int i = t; i < 2 * nq; i += FC_THREADS - 64) {
                const int k = ((i >> 1) * S + s) * 64 + (i & 1) * 32;
                if (k < K) prefetch_l2_keep(a.m + k);
            }
        }
        if (!a.in_rows) {  // (with a row map the rows are not known yet)
            constexpr int XL = (64 * (int)sizeof(XT) + 127) / 128;  // lines per row and block
            for (int i = t; i < nq * B * XL; i += FC_THREADS - 64) {
                const int l = i % XL, rb = i / XL, b = rb % B, q = rb / B;
                const int k = (q * S + s) * 64 + l * (128 / (int)sizeof(XT));
                if (k < K) prefetch_l2_keep(xg + (size_t)b * a.x_ld + k);
            }
        }
    }
    // The first ring of weight blocks is requested at once, by the thread that initialised the barriers and BEFORE the
    // wait for earlier work on the stream: the weights are constants of the layer (the interface requires them to be
    // complete when the call is issued), their addresses do not depend on the activations, and so the stream of this
    // call starts while the previous call is still finishing its columns - the memory system does not idle between
    // calls.  Everything else (x, m, tau, biases, row maps) is read after the wait.
    const int x0 = EPI == EPI_GLU ? tile * HALF : tile * TNT;
    const int x1 = EPI == EPI_GLU ? a.Nh + tile * HALF : tile * TNT + HALF;
    const int nq_first = nq < DS_NST ? nq : DS_NST;
    if (tid == 0) {
        for (int q = 0; q < nq_first; ++q) {
            mbar_arrive_expect_tx(&misc->wfull[q], DS_STAGE_W);
            const uint32_t dst = smem_u32(s_w) + q * DS_STAGE_W;
            tma_box_2d(dst, &tmap, x0, (q * S + s) * 64, &misc->wfull[q]);
            tma_box_2d(dst + DS_STAGE_W / 2, &tmap, x1, (q * S + s) * 64, &misc->wfull[q]);
        }
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&misc->tmem_base)), "r"(TNT) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    float bias0[2], bias1[2];

    griddep_wait();  // x, m, tau, the biases and the row maps may be outputs of the work just before this call
    griddep_launch_dependents();
    // x and m are read again by every column tile of the call (and m by every later call): ask L2 to keep them.
    const uint64_t pol_keep = a.l2_hints ? l2_policy_keep() : l2_policy_normal();
    // Only the thresholding warps need tau; each of their lanes asks for it here and first uses it after its first
    // activations have arrived, so the two round trips to L2 overlap.
    float tau = 0.0f;
    if constexpr (MODE == MODE_GATHER) {
        if (warp >= 2) tau = ld_act(a.tau);
    }
    prefetch_bias<BF16, EPI, TNT>(a, tile, s, per, bias0, bias1);
    if (a.in_rows && tid < 16) misc->rows[tid] = __ldcg(a.in_rows + (tid < B ? tid : 0));
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = misc->tmem_base;
    const uint32_t idesc = (1u << 4) | ((BF16 ? 1u : 0u) << 7) | ((BF16 ? 1u : 0u) << 10) | (0u << 15) | (1u << 16) |
                           ((uint32_t)(TNT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

    if (warp == 0) {
        // ---- TMA producer: two boxes per stage
        if (lane == 0) {
            int q = nq_first;  // the first ring went out above
            for (; q < nq; ++q) {
                const uint32_t st = (uint32_t)q % DS_NST;
                if (!mbar_wait(&misc->empty[st], (((uint32_t)q / DS_NST) & 1u) ^ 1u, 1, abort_flag, spin)) break;
                mbar_arrive_expect_tx(&misc->wfull[st], DS_STAGE_W);
                const int row0 = (q * S + s) * 64;
                const uint32_t dst = smem_u32(s_w) + st * DS_STAGE_W;
                tma_box_2d(dst, &tmap, x0, row0, &misc->wfull[st]);
                tma_box_2d(dst + DS_STAGE_W / 2, &tmap, x1, row0, &misc->wfull[st]);
            }
            // After a wait that ran out the MMA lane no longer consumes stages, but loads already issued still write
            // this CTA's shared memory: wait for them (fixed limit; they land within microseconds) before anyone leaves.
            if (*abort_flag) {
                int drain_abort = 0;
                for (int qq = q > DS_NST ? q - DS_NST : 0; qq < q; ++qq)
                    mbar_wait(&misc->wfull[(uint32_t)qq % DS_NST], ((uint32_t)qq / DS_NST) & 1u, 5, &drain_abort, TC_SPIN);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---- MMA issuer: per stage four MMAs of 16 rows
        if (lane == 0) {
            for (int q = 0; q < nq; ++q) {
                const uint32_t st = (uint32_t)q % DS_NST, par = ((uint32_t)q / DS_NST) & 1u;
                if (!mbar_wait(&misc->afull[st], par, 2, abort_flag, spin)) break;
                if (!mbar_wait(&misc->wfull[st], par, 2, abort_flag, spin)) break;
                tc_fence_after();
                misc->issued = 1;
#pragma unroll
                for (uint32_t kb = 0; kb < 4; ++kb) {
                    const uint64_t da = tc_desc(smem_u32(s_a) + st * ASTG + kb * BLK, LBO, 128, 0);
                    const uint64_t db = tc_desc(smem_u32(s_w) + st * DS_STAGE_W + kb * 2048, DS_STAGE_W / 2, 1024, 2);
                    tc_mma(tmem, da, db, idesc, (q > 0 || kb > 0) ? 1u : 0u);
                }
                tc_commit(&misc->empty[st]);
            }
            if (nq > 0 && !*abort_flag) tc_commit(&misc->done);
        }
        __syncwarp();
    } else {
        // ---- A operand: chunk jc = stage 2 q + half h; element (row r = part * B + b, position pos of the stage): block
        // pos / 16, K half (pos / 8) & 1, 8-row group r / 8, 16 bytes per row of the group, 2 bytes per position.
        // A lane takes ONE batch row and ROWS consecutive channels of the chunk (lane = channel group * ROWS + row): its
        // activations are one or two 16-byte loads, and the eight positions of a row inside a K half are one 16-byte
        // store per part.  (Rows of x that are not 16-byte aligned - K not a multiple of 8 - take scalar loads.)
        const int pw = warp - 2;
        constexpr int CPL = ROWS;                   // channels per lane
        constexpr int XV = CPL * (int)sizeof(XT) / 16;  // 16-byte loads of x per lane
        const int b = lane % ROWS, cgp = lane / ROWS, ch0 = cgp * CPL;
        const bool vec_ok = ((size_t)a.x_ld * sizeof(XT)) % 16 == 0;
        const int xrow = a.in_rows ? misc->rows[b < B ? b : 0] : (b < B ? b : 0);
        for (int jc = pw; jc < 2 * nq; jc += FC_WARPS - 2) {
            const int q = jc >> 1, h = jc & 1;
            const uint32_t st = (uint32_t)q % DS_NST;
            const int c = 2 * (q * S + s) + h;  // global 32-channel chunk
            const int k0 = c * 32 + ch0;        // this lane's first channel
            float xv[CPL], mv[CPL];
            if (vec_ok) {
                uint4 raw[XV];
#pragma unroll
                for (int v = 0; v < XV; ++v) {
                    const int kk = k0 + v * (16 / (int)sizeof(XT));
                    raw[v] = ld_act16_if(reinterpret_cast<const unsigned char *>(xg + (size_t)xrow * a.x_ld + kk), b < B && kk < K, pol_keep);
                }
                const XT *xe = reinterpret_cast<const XT *>(raw);
#pragma unroll
                for (int i = 0; i < CPL; ++i) xv[i] = widen1(xe[i]);
            } else {
#pragma unroll
                for (int i = 0; i < CPL; ++i) xv[i] = widen1(ld_act_if(xg + (size_t)xrow * a.x_ld + k0 + i, b < B && k0 + i < K));
            }
            if (K % 4 == 0) {
#pragma unroll
                for (int v = 0; v < CPL / 4; ++v) {
                    uint4 r4 = make_uint4(0, 0, 0, 0);
                    if (MODE == MODE_GATHER && a.m) r4 = ld_act16_if(reinterpret_cast<const unsigned char *>(a.m + k0 + 4 * v), b < B && k0 + 4 * v < K, pol_keep);
                    mv[4 * v] = __uint_as_float(r4.x); mv[4 * v + 1] = __uint_as_float(r4.y);
                    mv[4 * v + 2] = __uint_as_float(r4.z); mv[4 * v + 3] = __uint_as_float(r4.w);
                }
            } else {
#pragma unroll
                for (int i = 0; i < CPL; ++i) mv[i] = (MODE == MODE_GATHER && a.m) ? ld_act_if(a.m + k0 + i, b < B && k0 + i < K) : 0.0f;
            }
            bool go = true;
            if (lane == 0) go = mbar_wait(&misc->empty[st], (((uint32_t)q / DS_NST) & 1u) ^ 1u, 1, abort_flag, spin);
            go = __shfl_sync(0xffffffffu, go ? 1 : 0, 0) != 0;
            if (!go) break;
            uint32_t mine = 0;
            unsigned short part[CPL][3];
#pragma unroll
            for (int i = 0; i < CPL; ++i) {
                const float dv = (MODE == MODE_GATHER && a.m) ? __fsub_rn(xv[i], mv[i]) : xv[i];
                const bool kept = b < B && k0 + i < K && (MODE == MODE_DENSE || fabsf(dv) >= tau);
                mine |= kept ? (1u << i) : 0u;
                split_parts<BF16>(kept ? dv : 0.0f, part[i]);
            }
            if (b < B) {
#pragma unroll
                for (int v = 0; v < CPL / 8; ++v) {
                    const int pos = h * 32 + ch0 + 8 * v;   // first of eight consecutive positions: one K half of one block
                    unsigned char *dst = s_a + st * ASTG + (size_t)(pos >> 4) * BLK + ((pos >> 3) & 1) * LBO;
#pragma unroll
                    for (int p = 0; p < NSPLIT; ++p) {
                        const int r = p * B + b;
                        uint4 w;
                        w.x = (uint32_t)part[8 * v + 0][p] | ((uint32_t)part[8 * v + 1][p] << 16);
                        w.y = (uint32_t)part[8 * v + 2][p] | ((uint32_t)part[8 * v + 3][p] << 16);
                        w.z = (uint32_t)part[8 * v + 4][p] | ((uint32_t)part[8 * v + 5][p] << 16);
                        w.w = (uint32_t)part[8 * v + 6][p] | ((uint32_t)part[8 * v + 7][p] << 16);
                        *reinterpret_cast<uint4 *>(dst + (r >> 3) * 128 + (r & 7) * 16) = w;
                    }
                }
            }
            const unsigned bal = __reduce_or_sync(0xffffffffu, mine << ch0);   // union over the rows, all 32 channels
            if (MODE == MODE_GATHER && a.bits && tile == 0 && lane == 0 && c * 32 < K) a.bits[c] = bal;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(&misc->afull[st]);
        }
    }
    // ---- all threads: wait until the last MMA has finished
    if (nq > 0) mbar_wait(&misc->done, 0, 3, abort_flag, spin);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (*abort_flag && misc->issued) {  // MMAs issued before a wait ran out may still be writing the accumulator
        if (warp == 1 && lane == 0) tc_commit(&misc->done);
        __syncwarp();
        int drain_abort = 0;
        mbar_wait(&misc->done, 0, 4, &drain_abort, TC_SPIN);
    }
    const bool have_acc = nq > 0 && !*abort_flag;
    // Accumulator rows (part p of batch row b = row p B + b = TMEM lane) to shared memory.  A warp reaches the 32 lanes
    // of its quarter (warp mod 4), so warps 0 and 4 share lanes 0-31 and warps 1 and 5 lanes 32-63, half the columns each.
    if (have_acc && (warp & 3) * 32 < racc && (warp & 3) < 2) {
        const int lq = warp & 3;
#pragma unroll 1
        for (int c0 = (warp >> 2) * 64; c0 < (warp >> 2) * 64 + 64; c0 += 32) {
            uint32_t v[32];
            asm volatile(
                "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                  "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
                  "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
                  "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                : "r"(tmem + ((uint32_t)(lq * 32) << 16) + (uint32_t)c0));
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            const int r = lq * 32 + lane;
            if (r < racc) {
#pragma unroll
                for (int j = 0; j < 32; ++j) s_part[r * TC_PART_LD + c0 + j] = __uint_as_float(v[j]);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TNT) : "memory");
    // ---- cluster exchange, push form: the parts of an element are added (smallest first) and the sum goes straight to
    // the cluster rank that finishes its column - slot (this rank, row) of that rank's gather buffer - as an asynchronous
    // store that counts down the owner's barrier.  No cluster-wide barrier after the prologue: a rank finishes its columns
    // as soon as its own S partials are in, and may leave while its stores to the others are still under way.
    if (S > 1) cluster_wait();  // every rank's barrier is initialised (all ranks arrived before their streams)
    {
        // A thread keeps one column and walks the rows (two row phases per CTA), so owner, slot and the owner's
        // addresses are computed once.
        const int c = tid % TNT;
        int r, slot0, bstride;
        if constexpr (EPI == EPI_GLU) {
            const int j = c % HALF, hf = c / HALF;
            r = j / per;
            slot0 = (s * 16 * 2 + hf) * per + (j - r * per);
            bstride = 2 * per;
        } else {
            r = c / per;
            slot0 = s * 16 * per + (c - r * per);
            bstride = per;
        }
        const uint32_t dst0 = S > 1 ? cluster_addr(smem_addr(s_gather) + 4u * (uint32_t)slot0, (uint32_t)r) : 0u;
        const uint32_t dbar = S > 1 ? cluster_addr(recv_bar, (uint32_t)r) : 0u;
        for (int b = tid / TNT; b < B; b += FC_THREADS / TNT) {
            float v = 0.0f;
            if (have_acc) {
#pragma unroll
                for (int p = NSPLIT - 1; p >= 0; --p) v += s_part[(p * B + b) * TC_PART_LD + c];
            }
            if (S > 1) st_async_f32(dst0 + 4u * (uint32_t)(b * bstride), v, dbar);
            else s_gather[slot0 + b * bstride] = v;
        }
    }
    if (S > 1) {
        bool landed = false;
        for (uint32_t it = 0; it < (1u << 22) && !landed; ++it) landed = mbarrier_try_wait(recv_bar, 0);
        if (!landed) atomicCAS(&g_tc_status, 0, 6);  // never in a correct run; the result is then incomplete
    } else {
        __syncthreads();
    }
    finish_columns<BF16, 16, EPI, TNT>(a, tile, s, per, s_gather, bias0, bias1);
}

// ---- host side ------------------------------------------------------------------------------------------------

template <bool BF16, int ROWS, int MODE, typename XT, int EPI>
static cudaError_t launch_tc_r(const FcArgs &a, cudaStream_t st) {
    static SmemOptIn opt_in;
    auto kern = fc_tc_kernel<BF16, ROWS, MODE, XT, EPI>;
    cudaError_t e0 = ensure_dynamic_smem(kern, TC_SMEM, opt_in);
    if (e0 != cudaSuccess) return e0;
    return launch_cluster(kern, dim3(fc_tiles(a.Nh, EPI, TC_TN), a.S), dim3(FC_THREADS), TC_SMEM, a.S, st, g_tune.pdl != 0, a);
}

template <bool BF16, int MODE, typename XT, int EPI>
static cudaError_t launch_tc_t(const FcArgs &a, cudaStream_t st) {
    return a.B <= 8 ? launch_tc_r<BF16, 8, MODE, XT, EPI>(a, st) : launch_tc_r<BF16, 16, MODE, XT, EPI>(a, st);
}

template <bool BF16, int MODE, typename XT>
static cudaError_t launch_tc_e(int epi, const FcArgs &a, cudaStream_t st) {
    return epi == EPI_GLU ? launch_tc_t<BF16, MODE, XT, EPI_GLU>(a, st) : launch_tc_t<BF16, MODE, XT, EPI_BIAS>(a, st);
}

template <bool BF16>
static cudaError_t launch_tc_w(int mode, int xkind, int epi, const FcArgs &a, cudaStream_t st) {
    using ST = typename std::conditional<BF16, __nv_bfloat16, __half>::type;
    if (mode == MODE_DENSE)
        return xkind == 2 ? launch_tc_e<BF16, MODE_DENSE, float>(epi, a, st) : launch_tc_e<BF16, MODE_DENSE, ST>(epi, a, st);
    return xkind == 2 ? launch_tc_e<BF16, MODE_GATHER, float>(epi, a, st) : launch_tc_e<BF16, MODE_GATHER, ST>(epi, a, st);
}

// Resident CTAs: the occupancy queries count a kernel that allocates TMEM as one CTA per SM, but two CTAs with 128
// TMEM columns each do share an SM (measured), so the budget is the one of the FMA kernel, which has the same
// threads, registers and CTAs per SM.
static int tc_resident(int S) { return resident_ctas(S); }

static int tc_fills(int K, int S, int B, bool bf16) {
    const int cap_chunks = tc_cap_chunks(tc_groups(B, bf16 ? 3 : 2));
    return (((K + 31) / 32 + S - 1) / S + cap_chunks - 1) / cap_chunks;
}

// tune value 1 (default): calls whose kept channels fit the A-operand region in one fill per CTA - every further fill
// drains and refills the ring, and the mma.sync variants are then faster; 2: every batch 3..16 call.
bool tc_applicable(const FcArgs &a, int epi, bool bf16) {
    if (g_tune.tc == 0 || a.no_tc || a.B < 3 || a.B > 16 || a.ldw % 8 != 0 || !aligned16(a.W) || a.hold_dependents) return false;
    if (g_tune.tc >= 2) return true;
    if (a.B <= g_tune.fma_rows) return false;
    // ... and whose CTAs stream at least 32 chunks each: on shorter streams the heavier set-up (TMEM, barriers,
    // operand staging) of this kernel outweighs its gain (measured at K = N = 4096)
    const int S = tc_choose_split(a.K, a.Nh, epi, a.B, bf16);
    return tc_fills(a.K, S, a.B, bf16) == 1 && ((a.K + 31) / 32 + S - 1) / S >= 32;
}

// Split-K factor for the tensor-core kernel (tile width is fixed at 128): most CTAs that are all resident at
// once; ties: fewer fills of the A-operand region, then the smaller cluster.
int tc_choose_split(int K, int Nh, int epi, int B, bool bf16) {
    const int tiles = fc_tiles(Nh, epi, TC_TN);
    const int nchunks = (K + 31) / 32;
    const int cap_chunks = tc_cap_chunks(tc_groups(B, bf16 ? 3 : 2));
    int best_S = 1;
    long long best = -1;
    for (int S = 1; S <= MAX_CLUSTER; ++S) {
        if (g_tune.split_k > 0 && S > g_tune.split_k) continue;
        if (S > 1 && K / S < 64) continue;
        const long long ctas = (long long)tiles * S;
        if (S > 1 && ctas > tc_resident(S)) continue;
        const int fills = ((nchunks + S - 1) / S + cap_chunks - 1) / cap_chunks;
        // one more fill costs about as much as a tenth of the CTAs: prefer a single fill over the last few CTAs
        const long long score = (ctas > 2 * sm_count() ? 0 : ctas * 64) - (long long)(fills - 1) * 64 * 26;
        if (score > best) { best = score; best_S = S; }
    }
    return best_S;
}


// ---- dense-stream kernel: tensor map and launch ----------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static std::atomic<EncodeTiledFn> cached{nullptr};
    EncodeTiledFn fn = cached.load(std::memory_order_acquire);
    if (fn) return fn;
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess || !p) {
        cudaGetLastError();
        return nullptr;
    }
    fn = reinterpret_cast<EncodeTiledFn>(p);
    cached.store(fn, std::memory_order_release);
    return fn;
}

// W[K, ldw] of 16-bit elements as a 2-D tensor (columns innermost), boxes of 64 columns x 64 rows, 128-byte swizzle,
// rows and columns beyond the matrix read as zeros.  The map covers this GPU's own W only, and every box is copied to the one CTA that asked for it.
static bool ds_tensor_map(CUtensorMap *map, const void *W, int K, int ldw, bool bf16) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)ldw, (cuuint64_t)K};
    const cuuint64_t strides[1] = {(cuuint64_t)ldw * 2};
    const cuuint32_t box[2] = {64, 64};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(W), dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <bool BF16, int ROWS, int MODE, typename XT, int EPI>
static cudaError_t launch_ds_r(const FcArgs &a, const CUtensorMap &map, cudaStream_t st) {
    static SmemOptIn opt_in;
    auto kern = fc_ds_kernel<BF16, ROWS, MODE, XT, EPI>;
    cudaError_t e0 = ensure_dynamic_smem(kern, DS_SMEM, opt_in);
    if (e0 != cudaSuccess) return e0;
    return launch_cluster(kern, dim3(fc_tiles(a.Nh, EPI, TC_TN), a.S), dim3(FC_THREADS), DS_SMEM, a.S, st, g_tune.pdl != 0, a, map);
}
template <bool BF16, int MODE, typename XT, int EPI>
static cudaError_t launch_ds_t(const FcArgs &a, const CUtensorMap &map, cudaStream_t st) {
    return a.B <= 8 ? launch_ds_r<BF16, 8, MODE, XT, EPI>(a, map, st) : launch_ds_r<BF16, 16, MODE, XT, EPI>(a, map, st);
}
template <bool BF16, int MODE, typename XT>
static cudaError_t launch_ds_e(int epi, const FcArgs &a, const CUtensorMap &map, cudaStream_t st) {
    return epi == EPI_GLU ? launch_ds_t<BF16, MODE, XT, EPI_GLU>(a, map, st) : launch_ds_t<BF16, MODE, XT, EPI_BIAS>(a, map, st);
}
template <bool BF16>
static cudaError_t launch_ds_w(int mode, int xkind, int epi, const FcArgs &a, const CUtensorMap &map, cudaStream_t st) {
    using ST = typename std::conditional<BF16, __nv_bfloat16, __half>::type;
    if (mode == MODE_DENSE)
        return xkind == 2 ? launch_ds_e<BF16, MODE_DENSE, float>(epi, a, map, st) : launch_ds_e<BF16, MODE_DENSE, ST>(epi, a, map, st);
    return xkind == 2 ? launch_ds_e<BF16, MODE_GATHER, float>(epi, a, map, st) : launch_ds_e<BF16, MODE_GATHER, ST>(epi, a, map, st);
}

// tune "dense_stream": 0 never, 1 (default) batches above the fp32-FMA limit, 2 every batch 3..16 call.
bool ds_applicable(const FcArgs &a, int epi, bool bf16) {
    (void)epi; (void)bf16;
    if (g_tune.dense_stream == 0 || a.no_tc || a.B < 3 || a.B > 16 || a.ldw % 8 != 0 || !aligned16(a.W) || a.hold_dependents) return false;
    if (a.K < 64) return false;
    if (g_tune.dense_stream >= 2) return true;
    return a.B > g_tune.fma_rows;
}

// Split-K factor: the most CTAs (128-column tiles x S) that are all resident, at least one 64-row block per rank.
int ds_choose_split(int K, int Nh, int epi) {
    const int tiles = fc_tiles(Nh, epi, TC_TN), blocks = (K + 63) / 64;
    int best_S = 1;
    long long best = -1;
    for (int S = 1; S <= MAX_CLUSTER; ++S) {
        if (g_tune.split_k > 0 && S > g_tune.split_k) continue;
        if (S > blocks) continue;
        const long long ctas = (long long)tiles * S;
        if (S > 1 && ctas > tc_resident(S)) continue;
        if (ctas > best) { best = ctas; best_S = S; }
    }
    return best_S;
}

cudaError_t launch_fc_ds(bool bf16, int mode, int xkind, int epi, const FcArgs &a, cudaStream_t st) {
    CUtensorMap map;
    if (!ds_tensor_map(&map, a.W, a.K, a.ldw, bf16)) return cudaErrorNotSupported;
    return bf16 ? launch_ds_w<true>(mode, xkind, epi, a, map, st) : launch_ds_w<false>(mode, xkind, epi, a, map, st);
}

cudaError_t launch_fc_tc(bool bf16, int mode, int xkind, int epi, const FcArgs &a, cudaStream_t st) {
    return bf16 ? launch_tc_w<true>(mode, xkind, epi, a, st) : launch_tc_w<false>(mode, xkind, epi, a, st);
}

// Device address of the status word of the bounded waits, looked up once per device.
int *tc_status_ptr() {
    static std::atomic<int *> cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    if (dev >= 0 && dev < 64) {
        int *hit = cached[dev].load(std::memory_order_acquire);
        if (hit) return hit;
    }
    int *p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_tc_status) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    if (dev >= 0 && dev < 64) cached[dev].store(p, std::memory_order_release);
    return p;
}

// Reads and clears the status word of the bounded waits (synchronises the device).
int tc_take_status() {
    int v = 0, zero = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return -1; }
    if (cudaMemcpyFromSymbol(&v, g_tc_status, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return -1; }
    if (v) cudaMemcpyToSymbol(g_tc_status, &zero, sizeof(int));
    return v;
}

}  // namespace scap
