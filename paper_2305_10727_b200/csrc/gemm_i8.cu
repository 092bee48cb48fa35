// The fused layer kernel of libgpusq: INT8 GEMM on the 5th-generation tensor
// cores (tcgen05), 2:4-sparse or dense weight operand, INT32 accumulators in
// tensor memory, and the de-quantise / bias / GELU / convert epilogue.
//
// Orientation.  The layer is Y[M,N] = X[M,K] * W[N,K]^T.  tcgen05.mma.sp wants
// the sparse operand as MMA-A, so the kernel computes Y^T = W * X^T.
//
// CTA pairs.  Two CTAs on neighbouring SMs (a cluster of two) work on one
// output tile of 256 features x block_t tokens with cta_group::2 instructions:
//   MMA-M = 256: each CTA supplies its own 128 features of W (values and, for
//           the sparse variant, metadata) and keeps their accumulators in its
//           own tensor memory (one lane per feature);
//   MMA-N = block_t tokens (one 32-bit tensor-memory column each): each CTA
//           loads only half of the tile's activation rows, the instruction
//           reads both halves;
//   MMA-K = 64 (sparse) or 32 (dense) per instruction, 128 per pipeline stage.
// Sharing the activation tile halves the L2 -> shared-memory traffic per
// output and keeps the sparse instruction's operand reads within the
// shared-memory bandwidth of one SM.
//
// Persistent clusters (one per SM pair), twenty warps per CTA:
//   warp 0      TMA producer (one elected lane), in both CTAs; every load of a
//               stage counts its bytes on the full barrier of the pair's CTA 0
//   warp 1      tensor-memory owner (both CTAs); in CTA 0 one elected lane
//               issues the MMAs for the pair and signals barriers in both CTAs
//   warps 2-17  epilogue: each warp owns 16 tensor-memory lanes (features) and
//               every other 32-token chunk; four warps (64 features) fill one
//               staging tile per chunk.  The work on a chunk is short and
//               latency-bound, so several warps per scheduler are needed to
//               keep the issue slots busy
//   warps 18-19 one elected lane each issues the TMA stores of one 64-feature
//               half's staging tiles and recycles them
// Everything is handed over with mbarriers (full/empty per smem stage,
// full/empty per accumulator buffer, full/free per staging tile), so no warp
// waits for another one's instruction stream; two accumulator buffers let the
// epilogue of tile i overlap the main loop of tile i+1.
//
// FP16 epilogue: tcgen05.ld in the 16x256b (accumulator-fragment) shape with
// the next chunk's load in flight during the arithmetic, FP32 math, pairs of
// tokens packed to f16x2, stmatrix.trans into a 128-byte-swizzled
// [32 tokens][64 features] staging tile, TMA store to Y (full 128-byte row
// segments; rows beyond M and features beyond N clipped by the tensor map).
#include <cuda.h>
#include <cuda_fp16.h>

#include <atomic>
#include <mutex>

#include "common.cuh"
#include "ptx.cuh"
#include "quant_math.cuh"

namespace gpusq {

constexpr int kBlockF = 128;        // features per CTA and tile
constexpr int kPairF = 2 * kBlockF; // features per CTA pair and tile
constexpr int kBlockK = 128;        // K per stage
constexpr int kMaxBlockT = 224;     // tokens per tile (runtime value, multiple of 32)
constexpr int kChunkT = 32;         // tokens per epilogue chunk
// Chunk phases of the epilogue: eight epilogue warps per phase.  Two (16 warps of 96 registers) is
// what is built; one (8 warps) is as fast without GELU and slower with it or with INT8 output, three
// (24 warps of 72 registers, two staging tiles per group) is 1.5x slower on every layer.
#ifndef GPUSQ_PHASES
#define GPUSQ_PHASES 2
#endif
constexpr int kMaxPhases = 3;       // chunk phases: eight epilogue warps (128 features) per phase
constexpr int kTmemCols = 512;
constexpr int kAccStride = 256;     // column offset of the second accumulator
constexpr int kMetaCol = 224;       // metadata slots: 4 columns per stage from here (below the second accumulator)
constexpr int kMaxEpiGroups = 2 * kMaxPhases;   // groups of four epilogue warps: 64 features x chunk phase
constexpr int kMaxEpiBufs = 3;                  // staging tiles per group, at most
constexpr int kEpiBufBytes = kChunkT * 128;           // [32 tokens][64 features] f16

// kHalf: the FP16 2:4 sparse model (binary16 operands, FP32 accumulators) instead of INT8.  A stage
// still covers 128 columns of W: 128 bytes of kept values per feature row, and two 128-byte-swizzled
// activation tiles of 64 columns each, one behind the other.
template <bool kSparse, bool kHalf = false>
struct Cfg {
    static_assert(kSparse || !kHalf, "the FP16 model exists only in the 2:4 sparse form");
    static constexpr int kABytes = kHalf ? kBlockF * 128 : kSparse ? kBlockF * 64 : kBlockF * 128;
    static constexpr int kBAtoms = kHalf ? 2 : 1;                // 128-byte-wide activation tiles per stage
    static constexpr int kBBytes = kBAtoms * (kMaxBlockT / 2) * 128;   // this CTA's half of the token rows
    static constexpr int kMetaBytes = kSparse ? 2048 : 0;
    static constexpr int kStageBytes = kABytes + kBBytes + kMetaBytes;
    static constexpr int kStages = kHalf ? 4 : kSparse ? 7 : 5;
    // Epilogue warps: eight per chunk phase (the warps of phase p take the chunks c of a tile with
    // (p + tile count) mod kPhases == c mod kPhases).
    static constexpr int kPhases = kHalf ? 2 : GPUSQ_PHASES;
    static constexpr int kEpiWarps = 8 * kPhases;
    static constexpr int kStoreWarp0 = 2 + kEpiWarps;          // first of the two store warps
    static constexpr int kThreads = 32 * (kStoreWarp0 + 2);
    static constexpr int kEpiGroups = 2 * kPhases;             // 64 features x chunk phase: four warps share a staging tile
    static constexpr int kEpiBufs = kPhases == 3 ? 2 : kPhases == 1 ? 6 : kHalf ? 2 : 3;      // staging tiles per group
    static constexpr int kI8Bufs = 2 * kEpiBufs;               // INT8 output: one ring per phase over the same shared memory
    static constexpr int kEpiBytes = kEpiGroups * kEpiBufs * kEpiBufBytes;
    static constexpr int kCtlBytes = 1024;
    static constexpr int kSmemBytes = kStages * kStageBytes + kEpiBytes + kCtlBytes + 1024 /* alignment slack */;
    static constexpr int kMmasPerStage = kHalf ? 4 : kSparse ? 2 : 4;
    static constexpr int kAStepBytes = 32;                    // per MMA along K, all variants
    static constexpr int kBStepBytes = kHalf ? 64 : kSparse ? 64 : 32;
    static constexpr int kASwizzle = kHalf ? 128 : kSparse ? 64 : 128;
    static constexpr int kMetaColsPerMma = kHalf ? 1 : 2;     // 32-bit tensor-memory columns of metadata per MMA
    static_assert(kStageBytes % 1024 == 0, "stages keep the 1024-byte alignment of the swizzled tiles");
    static_assert(kStages <= 8, "eight metadata slots below the second accumulator");
    static_assert(kSmemBytes <= 232448, "shared memory per CTA");
};

struct Ctl {
    uint64_t full[8];
    uint64_t empty[8];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t drain;
    uint64_t stg_full[kMaxEpiGroups * kMaxEpiBufs];     // staging tile written by its four warps (flat: group * bufs + tile)
    uint64_t stg_free[kMaxEpiGroups * kMaxEpiBufs];     // staging tile read by its TMA store
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t wait_us;       // directly behind the flag: the bounded waits read their limit from here
};

struct GemmParams {
    const float *w_scale;
    const float *x_scale;
    const float *bias;
    const float *out_scale;
    void *Y;
    float *y_absmax;  // FP16 output only, nullable: max |Y| over the rounded outputs is merged into it
    int32_t *status;
    int64_t M;
    int N;
    int K;
    int block_t;    // tokens per tile, a multiple of 32: the height of the first n_big token tiles
    int n_big;      // token tiles of full height; the token tiles after them are 32 tokens lower
    int act;
    int out_type;
    int pair_cols;  // feature columns of 256 that are worked on as ordinary pair tiles
    int pair_tiles; // pair_cols x token tiles: tiles from here on are twin tiles of the last 128 features
    int num_tiles;
    int twin_n0;    // first feature of the twin column (256 pair_cols)
    int oob_row;    // a row coordinate beyond the weight tensor: loads from there fill with zeros
    uint32_t wait_us;   // limit of every device-side wait, microseconds
    int withhold;       // test hook: the first cluster's producers stop before the last k block of their first tile
};

// Where a tile sits.  Normally a pair shares `h` tokens and CTA `rank` owns 128 of the pair's 256
// features.  Token tiles come in two heights so that the number of tiles can be made to fit the
// number of CTA pairs (the last wave of a persistent launch is otherwise partly empty): the first
// n_big token tiles are block_t tokens high, the ones after them block_t - 32.
// When the last column of features is at most 128 wide (N mod 256 in 1..128: every
// layer of at most 128 features, and e.g. N = 384) that would leave the second CTA without output,
// so that column is worked on in "twin" tiles: each CTA owns the column's features of its OWN
// `block_t` tokens, and the pair's MMA runs over the k blocks twice, first against the token tile of
// CTA 0 with the weight block in CTA 0's shared memory and zeros in CTA 1's, then against CTA 1's
// tokens the other way round, so each CTA's accumulator ends up with W times its own tokens.
// Ordinary tiles come first (feature column fastest), twin tiles after them.
// kTwin = false (no twin column in this launch) compiles the test away.
template <bool kTwin>
struct TileWalk {
    int tile;       // cluster_id, cluster_id + num_clusters, ...
    int tn, tm;     // feature column and token tile of an ordinary tile, kept incrementally (no division per tile)
    int step_n, step_m;

    __device__ __forceinline__ TileWalk(const GemmParams &p, int cluster_id, int num_clusters)
    {
        const int cols = p.pair_cols > 0 ? p.pair_cols : 1;
        tile = cluster_id;
        tn = cluster_id % cols;
        tm = cluster_id / cols;
        step_n = num_clusters % cols;
        step_m = num_clusters / cols;
    }
    __device__ __forceinline__ void next(const GemmParams &p, int num_clusters)
    {
        tile += num_clusters;
        tn += step_n;
        tm += step_m;
        if (tn >= p.pair_cols) {
            tn -= p.pair_cols;
            ++tm;
        }
    }
    __device__ __forceinline__ bool twin(const GemmParams &p) const { return kTwin && tile >= p.pair_tiles; }
    // the tile is one of the lower ones (token tiles from n_big on)
    __device__ __forceinline__ bool low(const GemmParams &p) const { return !twin(p) && tm >= p.n_big; }
    // first feature and first token of CTA `rank`'s part, and the tile's height in tokens
    __device__ __forceinline__ void origin(const GemmParams &p, int rank, int &n0, int64_t &m0, int &h) const
    {
        if (twin(p)) {
            n0 = p.twin_n0;
            m0 = ((int64_t)(tile - p.pair_tiles) * 2 + rank) * p.block_t;
            h = p.block_t;
            return;
        }
        n0 = tn * kPairF + rank * kBlockF;
        const int below = tm - p.n_big;                 // > 0: that many lower tiles precede this one
        h = below >= 0 ? p.block_t - 32 : p.block_t;
        m0 = (int64_t)tm * p.block_t - (below > 0 ? (int64_t)below * 32 : 0);
    }
};

// A wait of this CTA expired: raise the abort flag in both CTAs of the pair and record where.
__device__ __forceinline__ void report_timeout(const GemmParams &p, Ctl *ctl, int tile, int role, int stage)
{
    const uint32_t flag = ptx::smem_u32(&ctl->abort_flag);
    const bool first = atomicExch(&ctl->abort_flag, 1u) == 0u;
    ptx::st_cluster_u32(ptx::map_to_cta(flag, ptx::cluster_ctarank() ^ 1u), 1u);
    if (first && p.status) {
        if (atomicCAS(p.status, 0, GPUSQ_ERR_TIMEOUT) == 0) {
            p.status[1] = tile;
            p.status[2] = role;
            p.status[3] = stage;
        }
    }
}

// Exact-erf GELU as GELU(y) = max(y, 0) - g(|y|), g(t) = t * Phi(-t) = t * 2^p(t) with
// p(t) = log2(Phi(-t)) a degree-6 polynomial on [0, 6] (gen_gelu_coeffs.py; |error| < 1.1e-5 in p up
// to t = 4.3, so g keeps a relative accuracy of ~8e-6 wherever the binary16 result is a normal
// number, negative tail included; beyond, where the result is subnormal, the fit is looser but stays
// within a fraction of the subnormal spacing).  Beyond t = 6, g < 2^-25.
// The polynomial is written in u = -t (odd coefficients negated), so that the result is one fused
// multiply-add max(y, 0) + u * 2^p.  The coefficients are duplicated so that a packed FP32
// instruction can take a pair straight from the constant bank.
__constant__ float2 kGeluC[7] = {
    {-1.000003934e+00f, -1.000003934e+00f}, {1.151062012e+00f, 1.151062012e+00f},
    {-4.591387510e-01f, -4.591387510e-01f}, {5.306138098e-02f, 5.306138098e-02f},
    {7.939796895e-03f, 7.939796895e-03f},   {7.468767581e-04f, 7.468767581e-04f},
    {3.226381159e-05f, 3.226381159e-05f},
};

__device__ __forceinline__ float ex2_approx(float x)
{
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// two values at a time: the polynomial runs on packed FP32 pairs (fma.rn.f32x2)
__device__ __forceinline__ float2 gelu_pair(float2 y)
{
    const float2 u = make_float2(fmaxf(-fabsf(y.x), -6.0f), fmaxf(-fabsf(y.y), -6.0f));
    float2 r = kGeluC[6];
#pragma unroll
    for (int d = 5; d >= 0; --d) r = __ffma2_rn(r, u, kGeluC[d]);
    // max(y, 0) + u * 2^p
    return __ffma2_rn(u, make_float2(ex2_approx(r.x), ex2_approx(r.y)),
                      make_float2(fmaxf(y.x, 0.0f), fmaxf(y.y, 0.0f)));
}

// FP16 epilogue of one worker warp.  The warp owns 16 tensor-memory lanes (features) and every
// other 32-token chunk of each tile.  Per chunk: wait for the chunk's tcgen05.ld (issued one chunk
// ahead), issue the next one, convert / scale / activate 16 values per thread, wait for a free
// staging tile, two stmatrix, proxy fence, arrive on the tile's full barrier.  The loop is written
// for few instructions per chunk: whatever can be precomputed or advanced incrementally is.
template <bool kAccFloat, int kBufs, int kPhases, bool kTwin>
struct EpiF16 {
    const GemmParams *p;
    Ctl *ctl;
    uint32_t tmem_base, stage0, stg_full0, stg_free0, tmem_empty0, tmem_empty1;
    float x_scale;
    int warp, lane, rank, cluster_id, num_clusters, tiles_n, num_tiles;

    // staging-tile ring of this warp's group
    uint32_t buf_addr, full_bar, free_bar, buf_idx, free_parity;
    uint32_t stm_off;          // this lane's stmatrix row address inside a staging tile (second one: + 2048)
    float2 sc2[2], bi2[2];     // scale and bias of this thread's two features, duplicated for packed math
    float amax;                // kAmax: largest |y| this thread has produced for a token that exists

    __device__ __forceinline__ void release(int acc)
    {
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive_cluster(acc ? tmem_empty1 : tmem_empty0);
    }

    // One chunk held in v (its load was issued earlier).  next_taddr != 0: issue this warp's next
    // load into vn; otherwise v was the warp's last chunk of the tile and the accumulator is released.
    // rows: tokens of the chunk that exist (32 except at the end of the tensor); only kAmax looks at
    // it, the stores clip by themselves.
    template <bool kGelu, bool kAmax>
    __device__ __forceinline__ bool step(uint32_t (&v)[16], uint32_t (&vn)[16], uint32_t next_taddr, int acc,
                                         int tile, int rows)
    {
        ptx::tmem_ld_wait_regs(v);
        if (next_taddr)
            ptx::tmem_ld_16x256b_x4(next_taddr, vn);
        else
            release(acc);
        uint32_t pk[8];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                // INT32 sums are converted; the FP16 model's FP32 sums are taken as they are (scale 1)
                const float2 a = kAccFloat ? make_float2(__uint_as_float(v[4 * i + 2 * j]), __uint_as_float(v[4 * i + 2 * j + 1]))
                                           : make_float2(__int2float_rn((int32_t)v[4 * i + 2 * j]),
                                                         __int2float_rn((int32_t)v[4 * i + 2 * j + 1]));
                float2 y = __ffma2_rn(a, sc2[j], bi2[j]);
                if (kGelu) y = gelu_pair(y);
                const __half2 hh = __floats2half2_rn(y.x, y.y);   // low = token 2(t%4), high = +1
                pk[2 * i + j] = *reinterpret_cast<const uint32_t *>(&hh);
                if (kAmax) {
                    // rounding is monotonic: the maximum of the rounded outputs is the rounded maximum.
                    // Rows past the end of the tensor hold the bias only and do not count.
                    const int tok = 8 * i + 2 * (lane & 3);
                    if (rows >= kChunkT) {
                        amax = fmaxf(amax, fmaxf(fabsf(y.x), fabsf(y.y)));
                    } else {
                        if (tok < rows) amax = fmaxf(amax, fabsf(y.x));
                        if (tok + 1 < rows) amax = fmaxf(amax, fabsf(y.y));
                    }
                }
            }
        // the staging tile's previous contents have been stored
        bool to;
        if (!ptx::mbar_wait_bounded(free_bar, free_parity, &ctl->abort_flag, to)) {
            if (to && lane == 0) report_timeout(*p, ctl, tile, 2, 200 + (int)buf_idx);
            return false;
        }
        // matrices of one stmatrix: (tokens 0-7, feat 0-7), (0-7, 8-15), (8-15, 0-7), (8-15, 8-15)
        ptx::stmatrix_x4_trans(buf_addr + stm_off, pk[0], pk[1], pk[2], pk[3]);
        ptx::stmatrix_x4_trans(buf_addr + stm_off + 2048u, pk[4], pk[5], pk[6], pk[7]);
        ptx::fence_proxy_async_smem();                     // this lane's writes, for the TMA store
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(full_bar);
        if (++buf_idx == (uint32_t)kBufs) {
            buf_idx = 0;
            free_parity ^= 1u;
            buf_addr = stage0;
            full_bar = stg_full0;
            free_bar = stg_free0;
        } else {
            buf_addr += kEpiBufBytes;
            full_bar += 8;
            free_bar += 8;
        }
        return true;
    }

    template <bool kGelu, bool kAmax>
    __device__ __forceinline__ void run()
    {
        const int quarter = warp & 3;                      // tensor-memory lanes [32q, 32q+32) are this warp's to read
        const int half = ((warp - 2) >> 2) & 1;            // which 16 of them
        const int par = (warp - 2) >> 3;                   // which chunks: every kPhases-th one
        const int nofs = quarter * 32 + 16 * half + (lane >> 2);       // this thread's first feature in the CTA's 128
        amax = 0.0f;
        {
            // stmatrix row of this lane: token 8 (mid / 2) + r of the tile, 16-byte column c16 (128-byte swizzle)
            const int mid = lane >> 3, r = lane & 7;
            const int tok = 8 * (mid >> 1) + r;
            const int c16 = 4 * (quarter & 1) + 2 * half + (mid & 1);
            stm_off = (uint32_t)(tok * 128 + ((c16 ^ r) << 4));
        }
        buf_addr = stage0;
        full_bar = stg_full0;
        free_bar = stg_free0;
        buf_idx = 0;
        free_parity = 1;                                   // first round: the tiles are free
        const int64_t M = p->M;
        const int N = p->N;
        const float *w_scale = p->w_scale, *bias = p->bias;

        // scale and bias of a tile are fetched one tile ahead: the loads are in flight during a whole tile
        float ws_next[2], bi_next[2];
        auto fetch = [&](const TileWalk<kTwin> &w) {
            int n0, unused_h;
            int64_t unused;
            w.origin(*p, rank, n0, unused, unused_h);
            const bool in = w.tile < num_tiles && n0 < N;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int n = n0 + nofs + 8 * j;           // N need not fill the last 128-feature block
                ws_next[j] = (in && n < N) ? (w_scale ? __ldg(w_scale + n) : 1.0f) : 0.0f;
                bi_next[j] = (in && n < N && bias) ? __ldg(bias + n) : 0.0f;
            }
        };
        TileWalk<kTwin> walk(*p, cluster_id, num_clusters);
        fetch(walk);
        int local = 0;
        for (; walk.tile < num_tiles; ++local) {
            const int tile = walk.tile;
            int n0, h;
            int64_t m0;
            walk.origin(*p, rank, n0, m0, h);
            walk.next(*p, num_clusters);
            const int acc = local & 1;
            const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
            const bool n_valid = n0 < N;                   // the pair's second CTA may lie past the last feature
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const float sc = __fmul_rn(ws_next[j], x_scale);
                sc2[j] = make_float2(sc, sc);
                bi2[j] = make_float2(bi_next[j], bi_next[j]);
            }
            fetch(walk);
            bool to;
            if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl->tmem_full[acc]), acc_phase, &ctl->abort_flag, to)) {
                if (to && lane == 0) report_timeout(*p, ctl, tile, 2, 100 + acc);
                return;
            }
            ptx::tc_fence_after();
            int nchunks = 0;
            if (n_valid) {
                const int64_t left = M - m0;               // > 0
                nchunks = left >= h ? h / kChunkT : (int)((left + kChunkT - 1) / kChunkT);
            }
            // this warp's chunks of the tile: c0, c0 + kPhases, ...; the phases rotate every tile
            const int c0 = (par + local) % kPhases;
            int mine = (nchunks - c0 + kPhases - 1) / kPhases;         // how many of them
            if (mine <= 0) {
                release(acc);
                continue;
            }
            uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32 + half * 16) << 16) +
                             (uint32_t)(acc * kAccStride + c0 * kChunkT);
            uint32_t v0[16], v1[16];
            ptx::tmem_ld_16x256b_x4(taddr, v0);
            // tokens that exist from this warp's chunk on (at least 32 everywhere but at the end of the tensor)
            const int64_t ahead = M - m0 - (int64_t)c0 * kChunkT;
            int rows = ahead > 4 * kMaxBlockT ? 4 * kMaxBlockT : (int)ahead;
            for (;;) {
                taddr += kPhases * kChunkT;
                if (!step<kGelu, kAmax>(v0, v1, --mine ? taddr : 0u, acc, tile, rows)) return;
                if (!mine) break;
                rows -= kPhases * kChunkT;
                taddr += kPhases * kChunkT;
                if (!step<kGelu, kAmax>(v1, v0, --mine ? taddr : 0u, acc, tile, rows)) return;
                if (!mine) break;
                rows -= kPhases * kChunkT;
            }
        }
        if (kAmax) {
            // largest |Y| of this warp as the binary16 value that was stored, merged as a bit pattern
            // (non-negative binary32 values order like their patterns)
            float m = __half2float(__float2half_rn(amax));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            if (lane == 0 && m > 0.0f) atomicMax(reinterpret_cast<unsigned int *>(p->y_absmax), __float_as_uint(m));
        }
    }
};

// INT8 epilogue of one worker warp (requantised output): the FP16 epilogue's structure with bytes.
// The warp owns 16 tensor-memory lanes (features) and every other 32-token chunk; tcgen05.ld in the
// 16x256b shape gives a thread, per block of eight tokens, two neighbouring tokens of features f and
// f + 8.  Their four codes, packed into one word, are exactly the fragment of the 8-bit matrix store
// (stmatrix m16n8 b8, transposed): one instruction per chunk writes the warp's 32 tokens x 16 features
// as 16-byte row pieces into a 128-byte-swizzled [32 tokens][128 features] staging tile that the
// eight warps of the same chunk parity fill together; a TMA store writes full 128-byte rows of Y.
template <int kI8Bufs, int kPhases, bool kTwin>
struct EpiI8 {
    const GemmParams *p;
    Ctl *ctl;
    uint8_t *epi_smem;
    uint32_t tmem_base, tmem_empty0, tmem_empty1;
    float x_scale, out_scale;
    int warp, lane, rank, cluster_id, num_clusters, tiles_n, num_tiles;

    uint32_t buf_addr, full_bar, free_bar, buf_idx, free_parity, ring0, full0, free0;
    uint32_t stm_off;
    float2 sc2[2], bi2[2];
    QuantScale qs;

    __device__ __forceinline__ void release(int acc)
    {
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive_cluster(acc ? tmem_empty1 : tmem_empty0);
    }

    template <bool kGelu>
    __device__ __forceinline__ bool step(uint32_t (&v)[16], uint32_t (&vn)[16], uint32_t next_taddr, int acc, int tile)
    {
        ptx::tmem_ld_wait_regs(v);
        if (next_taddr)
            ptx::tmem_ld_16x256b_x4(next_taddr, vn);
        else
            release(acc);
        uint32_t pk[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            // feature f: tokens 8i + 2(t%4), +1; feature f + 8: the same tokens
            float2 ya = __ffma2_rn(make_float2(__int2float_rn((int32_t)v[4 * i]), __int2float_rn((int32_t)v[4 * i + 1])), sc2[0], bi2[0]);
            float2 yb = __ffma2_rn(make_float2(__int2float_rn((int32_t)v[4 * i + 2]), __int2float_rn((int32_t)v[4 * i + 3])), sc2[1], bi2[1]);
            if (kGelu) {
                ya = gelu_pair(ya);
                yb = gelu_pair(yb);
            }
            // values beyond +-127 out_scale saturate: rare, so they are only detected here (one
            // compare per four values) and handled, clamp included, by the exact branch
            const bool beyond = fmaxf(fmaxf(fabsf(ya.x), fabsf(ya.y)), fmaxf(fabsf(yb.x), fabsf(yb.y))) > qs.x_max;
            uint32_t differ = 0;
            float2 ma = quant2_sums<false>(ya, qs, differ), mb = quant2_sums<false>(yb, qs, differ);
            if (differ != 0u || beyond || qs.always_divide) {
                ma = quant2_exact<true>(ya, qs);
                mb = quant2_exact<true>(yb, qs);
            }
            pk[i] = pack4_low_bytes(ma, mb);
        }
        bool to;
        if (!ptx::mbar_wait_bounded(free_bar, free_parity, &ctl->abort_flag, to)) {
            if (to && lane == 0) report_timeout(*p, ctl, tile, 2, 200 + (int)buf_idx);
            return false;
        }
        ptx::stmatrix_x4_trans_b8(buf_addr + stm_off, pk[0], pk[1], pk[2], pk[3]);
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(full_bar);
        if (++buf_idx == (uint32_t)kI8Bufs) {
            buf_idx = 0;
            free_parity ^= 1u;
            buf_addr = ring0;
            full_bar = full0;
            free_bar = free0;
        } else {
            buf_addr += kEpiBufBytes;
            full_bar += 8;
            free_bar += 8;
        }
        return true;
    }

    template <bool kGelu>
    __device__ __forceinline__ void run()
    {
        const int quarter = warp & 3;                      // tensor-memory lanes [32q, 32q+32) are this warp's to read
        const int half = ((warp - 2) >> 2) & 1;            // which 16 of them
        const int par = (warp - 2) >> 3;                   // which chunks: every kPhases-th one
        const int nofs = quarter * 32 + 16 * half + (lane >> 2);
        // this lane's address in the matrix store: row = token `lane` of the chunk, the warp's 16-byte column
        stm_off = (uint32_t)(lane * 128 + (((2 * quarter + half) ^ (lane & 7)) << 4));
        // the barriers of the staging tiles, taken as one array: ring `par` uses entries par * kI8Bufs ...
        ring0 = ptx::smem_u32(epi_smem + par * kI8Bufs * kEpiBufBytes);
        full0 = ptx::smem_u32(&ctl->stg_full[0]) + (uint32_t)(par * kI8Bufs * 8);
        free0 = ptx::smem_u32(&ctl->stg_free[0]) + (uint32_t)(par * kI8Bufs * 8);
        buf_addr = ring0;
        full_bar = full0;
        free_bar = free0;
        buf_idx = 0;
        free_parity = 1;                                   // first round: the tiles are free
        const int64_t M = p->M;
        const int N = p->N;
        const float *w_scale = p->w_scale, *bias = p->bias;
        qs = make_quant_scale(out_scale);

        float ws_next[2], bi_next[2];
        auto fetch = [&](const TileWalk<kTwin> &w) {
            int n0, unused_h;
            int64_t unused;
            w.origin(*p, rank, n0, unused, unused_h);
            const bool in = w.tile < num_tiles && n0 < N;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int n = n0 + nofs + 8 * j;
                ws_next[j] = (in && n < N) ? __ldg(w_scale + n) : 0.0f;
                bi_next[j] = (in && n < N && bias) ? __ldg(bias + n) : 0.0f;
            }
        };
        TileWalk<kTwin> walk(*p, cluster_id, num_clusters);
        fetch(walk);
        int local = 0;
        for (; walk.tile < num_tiles; ++local) {
            const int tile = walk.tile;
            int n0, h;
            int64_t m0;
            walk.origin(*p, rank, n0, m0, h);
            walk.next(*p, num_clusters);
            const int acc = local & 1;
            const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
            const bool n_valid = n0 < N;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const float sc = __fmul_rn(ws_next[j], x_scale);
                sc2[j] = make_float2(sc, sc);
                bi2[j] = make_float2(bi_next[j], bi_next[j]);
            }
            fetch(walk);
            bool to;
            if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl->tmem_full[acc]), acc_phase, &ctl->abort_flag, to)) {
                if (to && lane == 0) report_timeout(*p, ctl, tile, 2, 100 + acc);
                return;
            }
            ptx::tc_fence_after();
            int nchunks = 0;
            if (n_valid) {
                const int64_t left = M - m0;
                nchunks = left >= h ? h / kChunkT : (int)((left + kChunkT - 1) / kChunkT);
            }
            const int c0 = (par + local) % kPhases;
            int mine = (nchunks - c0 + kPhases - 1) / kPhases;
            if (mine <= 0) {
                release(acc);
                continue;
            }
            uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32 + half * 16) << 16) +
                             (uint32_t)(acc * kAccStride + c0 * kChunkT);
            uint32_t v0[16], v1[16];
            ptx::tmem_ld_16x256b_x4(taddr, v0);
            for (;;) {
                taddr += kPhases * kChunkT;
                if (!step<kGelu>(v0, v1, --mine ? taddr : 0u, acc, tile)) return;
                if (!mine) break;
                taddr += kPhases * kChunkT;
                if (!step<kGelu>(v1, v0, --mine ? taddr : 0u, acc, tile)) return;
                if (!mine) break;
            }
        }
    }
};

// kOut = GPUSQ_OUT_F16 / _I8 / _I32: one instantiation per output type, so that each epilogue gets its
// own register allocation
// kAmax: the FP16 epilogue also merges max |Y| into a device word (its own instantiation, so that the
// ordinary kernel's register allocation is untouched)
template <bool kSparse, int kOut, bool kHalf = false, bool kTwin = false, bool kAmax = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__((Cfg<kSparse, kHalf>::kThreads), 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_b2, const __grid_constant__ CUtensorMap map_e,
               const __grid_constant__ CUtensorMap map_y, const GemmParams p)
{
    using C = Cfg<kSparse, kHalf>;
    extern __shared__ uint8_t smem_raw[];
    // operand tiles need 1024-byte alignment for the 128-byte swizzle; both CTAs of a pair get the same offsets
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *epi_smem = smem + C::kStages * C::kStageBytes;
    Ctl *ctl = reinterpret_cast<Ctl *>(epi_smem + C::kEpiBytes);
    constexpr int kBufs = C::kEpiBufs;      // staging tiles per group in the FP16-output path
    constexpr int kPhases = C::kPhases, kEpiWarps = C::kEpiWarps, kStoreWarp0 = C::kStoreWarp0, kI8Bufs = C::kI8Bufs;
    volatile uint32_t *abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();            // 0 issues the MMAs of the pair
    const int cluster_id = blockIdx.x >> 1;
    const int num_clusters = gridDim.x >> 1;
    const int tiles_n = (p.N + kPairF - 1) / kPairF;
    const int num_tiles = p.num_tiles;
    const int k_blocks = (p.K + kBlockK - 1) / kBlockK;        // k blocks of the layer; a twin tile takes them twice

    auto a_smem = [&](int s) { return smem + s * C::kStageBytes; };
    auto b_smem = [&](int s) { return smem + s * C::kStageBytes + C::kABytes; };
    auto m_smem = [&](int s) { return smem + s * C::kStageBytes + C::kABytes + C::kBBytes; };

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&ctl->full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctl->empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(ptx::smem_u32(&ctl->tmem_full[a]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctl->tmem_empty[a]), 2 * kEpiWarps);   // the epilogue warps of both CTAs
        }
        ptx::mbar_init(ptx::smem_u32(&ctl->drain), 1);
        for (int g = 0; g < C::kEpiGroups * kBufs; ++g) {
            ptx::mbar_init(ptx::smem_u32(&ctl->stg_full[g]), kOut == GPUSQ_OUT_I8 ? 8 : 4);
            ptx::mbar_init(ptx::smem_u32(&ctl->stg_free[g]), 1);
        }
        ctl->abort_flag = 0;
        ctl->wait_us = p.wait_us;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&map_a);
        ptx::prefetch_tensormap(&map_b);
        if (p.n_big * p.pair_cols < p.pair_tiles) ptx::prefetch_tensormap(&map_b2);
        if (kSparse) ptx::prefetch_tensormap(&map_e);
        if (kOut != GPUSQ_OUT_I32) ptx::prefetch_tensormap(&map_y);
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(ptx::smem_u32(&ctl->tmem_base), kTmemCols);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync();            // the other CTA's barriers exist before anything is signalled on them
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    // Programmatic dependent launch: everything above ran while the previous kernel in the stream was
    // still finishing; its results (activations, their scale) may be read from here on.  The next
    // kernel in the stream may start its own set-up now.
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (ptx::elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            uint32_t issued = 0;            // bit s: a load into stage s was issued
            uint32_t last_parity = 0;       // bit s: parity of the last phase issued into stage s
            bool ok = true;
            for (TileWalk<kTwin> walk(p, cluster_id, num_clusters); ok && walk.tile < num_tiles; walk.next(p, num_clusters)) {
                const int tile = walk.tile;
                const bool twin = walk.twin(p);
                const int tw = tile - p.pair_tiles;                               // index among the twin tiles
                const int tn = twin ? 0 : walk.tn;
                const int num_kb = twin ? 2 * k_blocks : k_blocks;
                int n0_unused, h;
                int64_t m0;
                walk.origin(p, 0, n0_unused, m0, h);                               // token origin of the pair's tile
                const int half_t = h >> 1;
                const CUtensorMap *mb = h == p.block_t ? &map_b : &map_b2;         // box height = half the tile's tokens
                // bytes both CTAs together bring in per stage
                const uint32_t stage_tx = 2u * (uint32_t)(C::kABytes + C::kBAtoms * half_t * 128 + C::kMetaBytes);
                for (int ks = 0; ks < num_kb; ++ks) {
                    if (p.withhold && tile == 0 && ks == num_kb - 1) {
                        // planted failure (test hook): these loads never come, the MMA issuer's wait runs out
                        ok = false;
                        break;
                    }
                    // twin tiles: pass `seg` of the k blocks runs against the token tile of CTA `seg`, whose
                    // weights sit in that CTA only (the other one loads zeros from beyond the tensor)
                    const int seg = twin ? ks / k_blocks : 0;
                    const int kb = ks - seg * k_blocks;
                    const int w0 = twin ? p.twin_n0 : tn * kPairF + (int)rank * kBlockF;   // first weight row wanted
                    const int f0 = (twin && seg != (int)rank) ? p.oob_row : w0;          // first weight row loaded
                    const int t0 = (twin ? (2 * tw + seg) * p.block_t : (int)m0) + (int)rank * half_t;
                    bool to;
                    if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag, to)) {
                        if (to) report_timeout(p, ctl, tile, 0, stage);
                        ok = false;
                        break;
                    }
                    // all bytes of the stage, from both CTAs, are counted on CTA 0's barrier
                    const uint32_t bar = ptx::map_to_cta(ptx::smem_u32(&ctl->full[stage]), 0);
                    if (rank == 0) ptx::mbar_arrive_expect_tx(ptx::smem_u32(&ctl->full[stage]), stage_tx);
                    ptx::tma_load_2d_pair(ptx::smem_u32(a_smem(stage)), &map_a, bar,
                                          kb * (kHalf ? 128 : kSparse ? 64 : 128), f0);
                    if (kHalf) {
                        // 128 binary16 columns = two tiles of 128 bytes per token row
                        ptx::tma_load_2d_pair(ptx::smem_u32(b_smem(stage)), mb, bar, kb * 256, t0);
                        ptx::tma_load_2d_pair(ptx::smem_u32(b_smem(stage)) + (uint32_t)(half_t * 128), mb, bar,
                                              kb * 256 + 128, t0);
                    } else {
                        ptx::tma_load_2d_pair(ptx::smem_u32(b_smem(stage)), mb, bar, kb * kBlockK, t0);
                    }
                    if (kSparse) {
                        // 2 KB metadata block of (feature tile, k block) = 8 rows of 256 bytes
                        ptx::tma_load_2d_pair(ptx::smem_u32(m_smem(stage)), &map_e, bar, 0,
                                              ((w0 / kBlockF) * k_blocks + kb) * 8);
                    }
                    issued |= 1u << stage;
                    last_parity = (last_parity & ~(1u << stage)) | (phase << stage);
                    if (++stage == C::kStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
            if (*abort_flag && rank == 0) {
                // do not leave while bulk copies may still land in the pair's shared memory
                for (int s = 0; s < C::kStages; ++s) {
                    if (issued & (1u << s)) {
                        uint32_t none[2] = {0u, p.wait_us};
                        bool to;
                        (void)ptx::mbar_wait_bounded(ptx::smem_u32(&ctl->full[s]), (last_parity >> s) & 1u, none, to);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------- MMA issuer
        if (rank == 0 && ptx::elect_one()) {
            const uint32_t idesc_big = kHalf ? ptx::make_idesc_f16_sparse(kPairF, p.block_t)
                                             : ptx::make_idesc_i8(kPairF, p.block_t, kSparse);
            const uint32_t idesc_low = kHalf ? ptx::make_idesc_f16_sparse(kPairF, p.block_t - 32)
                                             : ptx::make_idesc_i8(kPairF, p.block_t - 32, kSparse);
            int stage = 0;
            uint32_t phase = 0;
            int local = 0;
            bool ok = true;
            for (TileWalk<kTwin> walk(p, cluster_id, num_clusters); ok && walk.tile < num_tiles;
                 walk.next(p, num_clusters), ++local) {
                const int tile = walk.tile;
                const int acc = local & 1;
                const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
                bool to;
                if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl->tmem_empty[acc]), acc_phase ^ 1u, abort_flag, to)) {
                    if (to) report_timeout(p, ctl, tile, 1, 100 + acc);
                    ok = false;
                    break;
                }
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kAccStride);
                const int num_kb = walk.twin(p) ? 2 * k_blocks : k_blocks;
                // a tile of lower height (the token tiles from n_big on) takes the narrower instruction
                const bool low = walk.low(p);
                const uint32_t idesc = low ? idesc_low : idesc_big;
                const int half_t = (low ? p.block_t - 32 : p.block_t) >> 1;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl->full[stage]), phase, abort_flag, to)) {
                        if (to) report_timeout(p, ctl, tile, 1, stage);
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t meta_t = tmem_base + (uint32_t)(kMetaCol + 4 * stage);
                    if (kSparse) {
                        ptx::tc_cp_128x128b_pair(meta_t, ptx::make_smem_desc(ptx::smem_u32(m_smem(stage)), 128, 0));
                    }
                    const uint64_t adesc = ptx::make_smem_desc(ptx::smem_u32(a_smem(stage)), C::kASwizzle * 8, C::kASwizzle);
                    const uint64_t bdesc = ptx::make_smem_desc(ptx::smem_u32(b_smem(stage)), 1024, 128);
#pragma unroll
                    for (int k = 0; k < C::kMmasPerStage; ++k) {
                        const uint64_t ad = adesc + (uint64_t)((k * C::kAStepBytes) >> 4);
                        // FP16 model: MMAs 0, 1 read the first activation tile of the stage, 2, 3 the second
                        const uint64_t bd = kHalf ? bdesc + (uint64_t)(((k & 1) * 64 + (k >> 1) * half_t * 128) >> 4)
                                                  : bdesc + (uint64_t)((k * C::kBStepBytes) >> 4);
                        const uint32_t accum = (kb | k) != 0 ? 1u : 0u;
                        // 16-bit operands: one metadata column per MMA, addressed as an even column plus
                        // the selector bit of the instruction descriptor for the odd one
                        if (kHalf)
                            ptx::tc_mma_sp_f16_pair(d_tmem, ad, bd, meta_t + (uint32_t)(k & ~1), idesc | (uint32_t)(k & 1),
                                                    accum);
                        else if (kSparse)
                            ptx::tc_mma_sp_i8_pair(d_tmem, ad, bd, meta_t + 2u * k, idesc, accum);
                        else
                            ptx::tc_mma_i8_pair(d_tmem, ad, bd, idesc, accum);
                    }
                    // the stage is reusable in both CTAs once these MMAs are done
                    ptx::tc_commit_pair(ptx::smem_u32(&ctl->empty[stage]), 3);
                    if (++stage == C::kStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (ok) ptx::tc_commit_pair(ptx::smem_u32(&ctl->tmem_full[acc]), 3);
            }
            if (*abort_flag) {
                // let every MMA issued so far retire before tensor memory is released
                ptx::tc_commit(ptx::smem_u32(&ctl->drain));
                uint32_t none[2] = {0u, p.wait_us};
                bool to;
                (void)ptx::mbar_wait_bounded(ptx::smem_u32(&ctl->drain), 0, none, to);
            }
        }
    } else if (warp >= kStoreWarp0) {
        // --------------------------------------------------------- TMA stores
        // One lane per 64-feature half: waits for a staging tile to be filled, stores it, and hands
        // tiles back to the epilogue warps once the stores have read them.
        if (kOut == GPUSQ_OUT_F16 && ptx::elect_one()) {
            const int fgroup = warp - kStoreWarp0;         // features [64 fgroup, 64 fgroup + 64) of the CTA's 128
            uint32_t filled[kMaxPhases] = {};              // staging tiles stored so far, per chunk phase
            uint32_t prev1 = 0, prev2 = 0;                 // free barriers of the last two stores (0 = none)
            int local = 0;
            bool ok = true;
            for (TileWalk<kTwin> walk(p, cluster_id, num_clusters); ok && walk.tile < num_tiles;
                 walk.next(p, num_clusters), ++local) {
                const int tile = walk.tile;
                int n0, h;
                int64_t m0;
                walk.origin(p, (int)rank, n0, m0, h);
                if (n0 >= p.N) continue;
                const int64_t left = p.M - m0;
                const int nchunks = left >= h ? h / kChunkT : (int)((left + kChunkT - 1) / kChunkT);
                for (int c = 0; c < nchunks; ++c) {
                    const int par = (c + kPhases - local % kPhases) % kPhases;     // the warps with (par + local) % kPhases == c % kPhases fill this chunk
                    const int gi = fgroup * kPhases + par;
                    const uint32_t count = filled[par];
                    const uint32_t b = count % kBufs;
                    bool to;
                    if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl->stg_full[gi * kBufs + (int)b]), (count / kBufs) & 1u,
                                                abort_flag, to)) {
                        if (to) report_timeout(p, ctl, tile, 3, gi * 8 + (int)b);
                        ok = false;
                        break;
                    }
                    ptx::tma_store_2d(&map_y, ptx::smem_u32(epi_smem + (gi * kBufs + (int)b) * kEpiBufBytes),
                                      n0 + fgroup * 64, (int32_t)(m0 + c * kChunkT));
                    ptx::tma_store_commit();
                    // all but the two newest stores have read their tiles: hand the third newest back
                    ptx::tma_store_wait_read<2>();
                    if (prev2) ptx::mbar_arrive(prev2);
                    prev2 = prev1;
                    prev1 = ptx::smem_u32(&ctl->stg_free[gi * kBufs + (int)b]);
                    ++filled[par];
                }
            }
            // the staging tiles must stay valid until the bulk stores have read them, and the
            // stores must be complete before the kernel ends
            ptx::tma_store_wait_all<0>();
        } else if (kOut == GPUSQ_OUT_I8 && ptx::elect_one()) {
            // INT8 output: a staging tile holds all 128 features of a chunk; every chunk phase has its
            // ring; this lane serves the rings of even (first store warp) or odd phases
            const int odd = warp - kStoreWarp0;
            const uint32_t full0 = ptx::smem_u32(&ctl->stg_full[0]), free0 = ptx::smem_u32(&ctl->stg_free[0]);
            uint32_t filled[kMaxPhases] = {};              // staging tiles stored so far, per ring
            uint32_t prev1 = 0, prev2 = 0;
            int local = 0;
            bool ok = true;
            for (TileWalk<kTwin> walk(p, cluster_id, num_clusters); ok && walk.tile < num_tiles;
                 walk.next(p, num_clusters), ++local) {
                const int tile = walk.tile;
                int n0, h;
                int64_t m0;
                walk.origin(p, (int)rank, n0, m0, h);
                if (n0 >= p.N) continue;
                const int64_t left = p.M - m0;
                const int nchunks = left >= h ? h / kChunkT : (int)((left + kChunkT - 1) / kChunkT);
                for (int c = 0; c < nchunks; ++c) {
                    const int ring = (c + kPhases - local % kPhases) % kPhases;
                    if ((ring & 1) != odd) continue;
                    const uint32_t count = filled[ring];
                    const uint32_t slot = (uint32_t)(ring * kI8Bufs) + count % kI8Bufs;
                    bool to;
                    if (!ptx::mbar_wait_bounded(full0 + 8u * slot, (count / kI8Bufs) & 1u, abort_flag, to)) {
                        if (to) report_timeout(p, ctl, tile, 3, (int)slot);
                        ok = false;
                        break;
                    }
                    ptx::tma_store_2d(&map_y, ptx::smem_u32(epi_smem + (int)slot * kEpiBufBytes), n0,
                                      (int32_t)(m0 + c * kChunkT));
                    ptx::tma_store_commit();
                    ptx::tma_store_wait_read<2>();
                    if (prev2) ptx::mbar_arrive(prev2);
                    prev2 = prev1;
                    prev1 = free0 + 8u * slot;
                    ++filled[ring];
                }
            }
            ptx::tma_store_wait_all<0>();
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int quarter = warp & 3;                      // tensor-memory lanes [32q, 32q+32) are this warp's to read
        const int par = (warp - 2) >> 3;                   // FP16 path: which chunks, every other one
        const float x_scale = (kOut == GPUSQ_OUT_I32 || kHalf) ? 1.0f : __ldg(p.x_scale);
        const float out_scale = (kOut == GPUSQ_OUT_I8) ? __ldg(p.out_scale) : 1.0f;
        // the accumulators of both CTAs are released on CTA 0's barrier, where the MMA issuer waits
        const uint32_t tmem_empty0 = ptx::map_to_cta(ptx::smem_u32(&ctl->tmem_empty[0]), 0);
        const uint32_t tmem_empty1 = ptx::map_to_cta(ptx::smem_u32(&ctl->tmem_empty[1]), 0);
        const int group = (quarter >> 1) * kPhases + par;  // 64 features x chunk phase: the warps sharing staging tiles
        const uint32_t stage0 = ptx::smem_u32(epi_smem + group * kBufs * kEpiBufBytes);
        int local = 0;

        if (kOut == GPUSQ_OUT_F16) {
            EpiF16<kHalf, kBufs, kPhases, kTwin> e;
            e.p = &p;
            e.ctl = ctl;
            e.tmem_base = tmem_base;
            e.stage0 = stage0;
            e.stg_full0 = ptx::smem_u32(&ctl->stg_full[group * kBufs]);
            e.stg_free0 = ptx::smem_u32(&ctl->stg_free[group * kBufs]);
            e.tmem_empty0 = tmem_empty0;
            e.tmem_empty1 = tmem_empty1;
            e.x_scale = x_scale;
            e.warp = warp;
            e.lane = lane;
            e.rank = (int)rank;
            e.cluster_id = cluster_id;
            e.num_clusters = num_clusters;
            e.tiles_n = tiles_n;
            e.num_tiles = num_tiles;
            if (p.act == GPUSQ_ACT_GELU)
                e.template run<true, kAmax>();
            else
                e.template run<false, kAmax>();
        } else if (kOut == GPUSQ_OUT_I8) {
            EpiI8<kI8Bufs, kPhases, kTwin> e;
            e.p = &p;
            e.ctl = ctl;
            e.epi_smem = epi_smem;
            e.tmem_base = tmem_base;
            e.tmem_empty0 = tmem_empty0;
            e.tmem_empty1 = tmem_empty1;
            e.x_scale = x_scale;
            e.out_scale = out_scale;
            e.warp = warp;
            e.lane = lane;
            e.rank = (int)rank;
            e.cluster_id = cluster_id;
            e.num_clusters = num_clusters;
            e.tiles_n = tiles_n;
            e.num_tiles = num_tiles;
            if (p.act == GPUSQ_ACT_GELU)
                e.template run<true>();
            else
                e.template run<false>();
        } else {
            // raw INT32 accumulators (for bit-exact comparison): plain coalesced stores; the four warps
            // of a quarter take every fourth 16-token chunk
            for (TileWalk<kTwin> walk(p, cluster_id, num_clusters); walk.tile < num_tiles; walk.next(p, num_clusters), ++local) {
                const int tile = walk.tile;
                int n0, h;
                int64_t m0;
                walk.origin(p, (int)rank, n0, m0, h);
                const int acc = local & 1;
                const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
                const bool n_valid = n0 < p.N;
                const int n = n0 + quarter * 32 + lane;                // this thread's output feature
                bool to;
                if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl->tmem_full[acc]), acc_phase, abort_flag, to)) {
                    if (to && lane == 0) report_timeout(p, ctl, tile, 2, 100 + acc);
                    break;
                }
                ptx::tc_fence_after();
                const uint32_t tbase = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * kAccStride);
                for (int c = (warp - 2) >> 2; c < h / 16 && n_valid; c += kEpiWarps / 4) {
                    if (m0 + c * 16 >= p.M) break;
                    uint32_t r[16];
                    ptx::tmem_ld_32x32b_x16(tbase + (uint32_t)(c * 16), r);
                    ptx::tmem_ld_wait_regs(r);
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int64_t m = m0 + c * 16 + j;
                        if (m < p.M && n < p.N) reinterpret_cast<int32_t *>(p.Y)[m * p.N + n] = (int32_t)r[j];
                    }
                }
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(acc ? tmem_empty1 : tmem_empty0);
            }
        }
    }

    // neither CTA leaves while the other may still signal its barriers or read its shared memory
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(f);
    });
    return fn;
}

// 2-D row-major byte matrix [rows, row_bytes]; box = [box_rows, box_bytes]
static bool make_map_u8(CUtensorMap *map, const void *base, uint64_t rows, uint64_t row_bytes,
                        uint32_t box_bytes, uint32_t box_rows, CUtensorMapSwizzle swz)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {row_bytes, rows};
    cuuint64_t strides[1] = {row_bytes};
    cuuint32_t box[2] = {box_bytes, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Y [M, N] f16 row-major; box = 64 features x 32 tokens, 128-byte swizzle (the staging-tile layout)
static bool make_map_y_f16(CUtensorMap *map, void *base, uint64_t M, uint64_t N)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {N, M};
    cuuint64_t strides[1] = {N * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)kChunkT};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
           CUDA_SUCCESS;
}

// testing hooks (gpusq_testing.h): a forced tile height, and a forced number of full-height token tiles
static std::atomic<int> g_block_t_override{0};
static std::atomic<int> g_n_big_override{-1};
static std::atomic<unsigned> g_wait_us{ptx::kDefaultWaitUs};
static std::atomic<int> g_withhold_loads{0};
static std::atomic<int> g_cluster_cap{0};           // CTA pairs a launch may use (0 = as many as fit)

// How the token axis is cut into tiles: tok_tiles token tiles, the first n_big of them block_t tokens
// high, the others block_t - 32.
struct TilePlan {
    int block_t, n_big, tok_tiles;
};

// Relative time of one tile of h tokens over kb 128-wide k blocks.  Per tile and CTA the shared memory
// moves, per k block, 128 bytes per token (activations written and read) plus a fixed ~20 KB for the
// weight block (as much as 160 tokens), and the epilogue's staging costs as much as four k blocks per
// token: time per tile ~ (kb + 4) * h + 160 * kb.
static double tile_cost(double kb, int64_t h) { return (kb + 4.0) * (double)h + 160.0 * kb; }

// Time until the last cluster is done when cluster c works on tiles c, c + clusters, ...: the pair
// tiles (token tile major, pair_cols feature columns each) first, then the twin tiles of a last
// narrow feature column (two token tiles of block_t each, the k blocks taken twice).
static double makespan(const TilePlan &t, int64_t M, int pair_cols, bool twin_col, int clusters, double kb)
{
    double load[148] = {};
    const int C = clusters < 148 ? clusters : 148;
    int64_t i = 0;
    for (int tm = 0; tm < t.tok_tiles; ++tm) {
        const int low = tm - t.n_big;
        const int64_t h = low >= 0 ? t.block_t - 32 : t.block_t;
        const int64_t m0 = (int64_t)tm * t.block_t - (low > 0 ? (int64_t)low * 32 : 0);
        const double c = tile_cost(kb, M - m0 < h ? M - m0 : h);
        for (int tn = 0; tn < pair_cols; ++tn, ++i) load[i % C] += c;
    }
    if (twin_col) {
        const int64_t twins = ceil_div(M, 2 * (int64_t)t.block_t);
        for (int64_t w = 0; w < twins; ++w, ++i) load[i % C] += tile_cost(2.0 * kb, t.block_t);
    }
    double worst = 0.0;
    for (int c = 0; c < C; ++c) worst = load[c] > worst ? load[c] : worst;
    return worst;
}

// Tile heights for a launch.  Uniform tiles leave the last wave of the persistent launch partly
// empty whenever the tile count is not close to a multiple of the number of clusters (171 tiles on
// 74 clusters: three waves for 2.3 waves of work); mixing two heights 32 tokens apart gives a tile
// count that fits.  Searched only while the launch has few waves (beyond that the last wave weighs
// little and uniform tiles of the best height are taken); the result is remembered per shape.
static TilePlan plan_tiles(int64_t M, int pair_cols, bool twin_col, int clusters, int K)
{
    const double kb = (double)ceil_div(K, kBlockK);
    const int forced = g_block_t_override.load(std::memory_order_relaxed);
    const int forced_big = g_n_big_override.load(std::memory_order_relaxed);
    if (forced) {
        TilePlan t = {forced, (int)ceil_div(M, forced), (int)ceil_div(M, forced)};
        if (forced_big >= 0 && forced >= 64 && pair_cols > 0) {
            // as many full-height tiles as asked for (at most what covers M), lower ones for the rest
            const int64_t nb = forced_big < ceil_div(M, forced) ? forced_big : ceil_div(M, forced);
            const int64_t rest = M - nb * forced;
            t.n_big = (int)nb;
            t.tok_tiles = (int)(nb + (rest > 0 ? ceil_div(rest, forced - 32) : 0));
        }
        return t;
    }
    struct Entry {
        int64_t M;
        int pair_cols, twin, clusters, K;
        TilePlan plan;
    };
    static std::mutex mu;
    static Entry cache[64];
    static int used = 0, next = 0;
    {
        std::lock_guard<std::mutex> lock(mu);
        for (int i = 0; i < used; ++i)
            if (cache[i].M == M && cache[i].pair_cols == pair_cols && cache[i].twin == (int)twin_col &&
                cache[i].clusters == clusters && cache[i].K == K)
                return cache[i].plan;
    }
    TilePlan best = {kMaxBlockT, 0, 0};
    double best_cost = 1e300;
    auto consider = [&](const TilePlan &t) {
        const double c = makespan(t, M, pair_cols, twin_col, clusters, kb);
        if (c < best_cost * 0.999) {
            best_cost = c;
            best = t;
        }
    };
    for (int bt = kMaxBlockT; bt >= 32; bt -= 32) {
        const int64_t t_min = ceil_div(M, bt);
        if (t_min > 0x7FFFFFF) continue;
        consider({bt, (int)t_min, (int)t_min});                            // uniform
        if (bt < 64 || pair_cols == 0 || t_min * pair_cols > 16 * (int64_t)clusters) continue;
        const int64_t t_max = ceil_div(M, bt - 32);
        for (int64_t T = t_min; T < t_max; ++T) {
            // fewest full-height tiles with which T tiles cover M
            const int64_t need = M - T * (bt - 32);
            const int64_t nb = need > 0 ? ceil_div(need, 32) : 0;
            if (nb > T) continue;
            consider({bt, (int)nb, (int)T});
        }
    }
    std::lock_guard<std::mutex> lock(mu);
    cache[next] = {M, pair_cols, (int)twin_col, clusters, K, best};
    next = (next + 1) % 64;
    used = used < 64 ? used + 1 : 64;
    return best;
}

// Fills the tiling fields of the parameters; false when the tile count does not fit 31 bits.
static bool set_tiling(GemmParams &p, int64_t M, int N, int K_cost, int clusters)
{
    const int tiles_n = (N + kPairF - 1) / kPairF;
    // a last feature column of at most 128 features is worked on in twin tiles (see TileWalk)
    const bool twin_col = N - (tiles_n - 1) * kPairF <= kBlockF && M < 0x7FFFFFFF - 4 * kMaxBlockT;
    p.pair_cols = twin_col ? tiles_n - 1 : tiles_n;
    TilePlan t;
    if (p.pair_cols == 0) {
        // twin tiles only: each cluster takes two token tiles and the k blocks twice
        t = plan_tiles(ceil_div(M, 2), 1, false, clusters, 2 * K_cost);
        t = {t.block_t, 0, 0};
    } else {
        t = plan_tiles(M, p.pair_cols, twin_col, clusters, K_cost);
    }
    p.block_t = t.block_t;
    p.n_big = t.n_big;
    const int64_t pair_tiles = (int64_t)p.pair_cols * t.tok_tiles;
    const int64_t tiles = pair_tiles + (twin_col ? ceil_div(M, 2 * (int64_t)t.block_t) : 0);
    if (tiles > 0x7FFFFFFF) return false;
    p.pair_tiles = (int)pair_tiles;
    p.num_tiles = (int)tiles;
    p.twin_n0 = p.pair_cols * kPairF;
    p.oob_row = round_up(N, kPairF);  // beyond the packed rows (N rounded up) and the plain ones (N) alike
    p.wait_us = g_wait_us.load(std::memory_order_relaxed);
    p.withhold = g_withhold_loads.load(std::memory_order_relaxed);
    return true;
}

// SM pairs that can hold one cluster of this kernel each, per device (0 = unknown yet)
template <bool kSparse, bool kHalf = false>
static int max_clusters(int sms)
{
    static std::mutex mu;
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return sms / 2;
    std::lock_guard<std::mutex> lock(mu);
    if (cached[dev] == 0) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(sms & ~1), 1, 1);
        cfg.blockDim = dim3(Cfg<kSparse, kHalf>::kThreads, 1, 1);
        cfg.dynamicSmemBytes = Cfg<kSparse, kHalf>::kSmemBytes;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, gemm_i8_kernel<kSparse, GPUSQ_OUT_F16, kHalf>, &cfg) != cudaSuccess || n <= 0) {
            (void)cudaGetLastError();
            n = sms / 2;
        }
        cached[dev] = n < sms / 2 ? n : sms / 2;
    }
    return cached[dev];
}

// measurement hook (gpusq_testing.h): fewer CTA pairs than fit
static int capped(int clusters)
{
    const int cap = g_cluster_cap.load(std::memory_order_relaxed);
    return cap > 0 && cap < clusters ? cap : clusters;
}

// The kernels need more dynamic shared memory than the default limit; the attribute is per device.
template <typename F>
static bool allow_smem(F kernel, int bytes)
{
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
}

// once per device and operand kind (0 sparse INT8, 1 dense INT8, 2 sparse FP16)
static bool prepare_device(int kind)
{
    static std::mutex mu;
    static uint8_t done[64][3] = {};       // 1 = set, 2 = failed
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    std::lock_guard<std::mutex> lock(mu);
    if (done[dev][kind] == 0) {
        bool ok = true;
        if (kind == 0) {
            const int b = Cfg<true>::kSmemBytes;
            ok = allow_smem(gemm_i8_kernel<true, GPUSQ_OUT_F16>, b) && allow_smem(gemm_i8_kernel<true, GPUSQ_OUT_I8>, b) &&
                 allow_smem(gemm_i8_kernel<true, GPUSQ_OUT_I32>, b) &&
                 allow_smem(gemm_i8_kernel<true, GPUSQ_OUT_F16, false, true>, b) &&
                 allow_smem(gemm_i8_kernel<true, GPUSQ_OUT_I8, false, true>, b) &&
                 allow_smem(gemm_i8_kernel<true, GPUSQ_OUT_I32, false, true>, b) &&
                 allow_smem(gemm_i8_kernel<true, GPUSQ_OUT_F16, false, false, true>, b) &&
                 allow_smem(gemm_i8_kernel<true, GPUSQ_OUT_F16, false, true, true>, b);
        } else if (kind == 1) {
            const int b = Cfg<false>::kSmemBytes;
            ok = allow_smem(gemm_i8_kernel<false, GPUSQ_OUT_F16>, b) && allow_smem(gemm_i8_kernel<false, GPUSQ_OUT_I8>, b) &&
                 allow_smem(gemm_i8_kernel<false, GPUSQ_OUT_I32>, b) &&
                 allow_smem(gemm_i8_kernel<false, GPUSQ_OUT_F16, false, true>, b) &&
                 allow_smem(gemm_i8_kernel<false, GPUSQ_OUT_I8, false, true>, b) &&
                 allow_smem(gemm_i8_kernel<false, GPUSQ_OUT_I32, false, true>, b);
        } else {
            const int b = Cfg<true, true>::kSmemBytes;
            ok = allow_smem(gemm_i8_kernel<true, GPUSQ_OUT_F16, true>, b) && allow_smem(gemm_i8_kernel<true, GPUSQ_OUT_I32, true>, b) &&
                 allow_smem(gemm_i8_kernel<true, GPUSQ_OUT_F16, true, true>, b) &&
                 allow_smem(gemm_i8_kernel<true, GPUSQ_OUT_I32, true, true>, b);
        }
        if (!ok) (void)cudaGetLastError();
        done[dev][kind] = ok ? 1 : 2;
    }
    return done[dev][kind] == 1;
}

template <typename Kernel>
static int launch_on(Kernel kernel, int threads, int smem_bytes, const CUtensorMap &map_a, const CUtensorMap &map_b,
                     const CUtensorMap &map_b2, const CUtensorMap &map_e, const CUtensorMap &map_y,
                     const GemmParams &p, int clusters, void *stream)
{
    const int grid = 2 * (p.num_tiles < clusters ? p.num_tiles : clusters);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = (cudaStream_t)stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // start while the previous kernel drains
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kernel, map_a, map_b, map_b2, map_e, map_y, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return GPUSQ_ERR_CUDA;
    }
    return GPUSQ_OK;
}

template <bool kSparse>
static int launch_gemm(const int8_t *Xq, const void *Wsrc, const float *w_scale, const float *x_scale,
                       const float *bias, int act, int out_type, const float *out_scale, void *Y, int64_t M,
                       int N, int K, int32_t *status_buf, void *stream, float *y_absmax = nullptr)
{
    using C = Cfg<kSparse>;
    if (!Xq || !Wsrc || !Y) return GPUSQ_ERR_NULL;
    if (out_type < 0 || out_type > 2 || act < 0 || act > 1) return GPUSQ_ERR_ARG;
    if (out_type != GPUSQ_OUT_I32 && (!w_scale || !x_scale)) return GPUSQ_ERR_NULL;
    if (out_type == GPUSQ_OUT_I8 && !out_scale) return GPUSQ_ERR_NULL;
    if (M <= 0 || N <= 0 || K <= 0 || K % 16 || M > 0x7FFFFFFF) return GPUSQ_ERR_SHAPE;
    // rows of Y are written by bulk tensor stores, whose row pitch is a multiple of 16 bytes
    if ((out_type == GPUSQ_OUT_F16 && N % 8) || (out_type == GPUSQ_OUT_I8 && N % 16)) return GPUSQ_ERR_SHAPE;
    if (!aligned(Xq, 16) || !aligned(Wsrc, 16) || !aligned(Y, 16)) return GPUSQ_ERR_ALIGN;
    if (int st = check_arch()) return st;
    if (!prepare_device(kSparse ? 0 : 1)) return GPUSQ_ERR_CUDA;

    const int sms = num_sms();
    const int clusters = capped(max_clusters<kSparse>(sms));
    if (clusters <= 0) return GPUSQ_ERR_CUDA;

    GemmParams p;
    p.w_scale = w_scale;
    p.x_scale = x_scale;
    p.bias = bias;
    p.out_scale = out_scale;
    p.Y = Y;
    p.y_absmax = y_absmax;
    p.status = status_buf;
    p.M = M;
    p.N = N;
    p.K = K;
    p.act = act;
    p.out_type = out_type;
    if (!set_tiling(p, M, N, K, clusters)) return GPUSQ_ERR_SHAPE;
    const bool twin_col = p.pair_tiles < p.num_tiles;
    const bool mixed = p.block_t >= 64;      // the lower height exists
    const int Kp = round_up(K, 128), Np = round_up(N, kPairF);

    CUtensorMap map_a, map_b;
    bool ok;
    if (kSparse)
        ok = make_map_u8(&map_a, Wsrc, (uint64_t)Np, (uint64_t)Kp / 2, 64, kBlockF, CU_TENSOR_MAP_SWIZZLE_64B);
    else
        ok = make_map_u8(&map_a, Wsrc, (uint64_t)N, (uint64_t)K, 128, kBlockF, CU_TENSOR_MAP_SWIZZLE_128B);
    ok = ok && make_map_u8(&map_b, Xq, (uint64_t)M, (uint64_t)K, 128, (uint32_t)(p.block_t / 2),
                           CU_TENSOR_MAP_SWIZZLE_128B);
    CUtensorMap map_b2 = map_b;     // the activation box of the lower tiles
    if (mixed)
        ok = ok && make_map_u8(&map_b2, Xq, (uint64_t)M, (uint64_t)K, 128, (uint32_t)(p.block_t / 2 - 16),
                               CU_TENSOR_MAP_SWIZZLE_128B);
    CUtensorMap map_e = map_b;      // placeholder unless the weight is sparse
    if (kSparse) {
        // metadata blocks of 2 KB, viewed as 8 rows of 256 bytes each
        const uint8_t *meta = reinterpret_cast<const uint8_t *>(Wsrc) + (size_t)Np * (Kp / 2);
        ok = ok && make_map_u8(&map_e, meta, (uint64_t)(Np / 128) * (Kp / 128) * 8, 256, 256, 8,
                               CU_TENSOR_MAP_SWIZZLE_NONE);
    }
    CUtensorMap map_y = map_b;      // placeholder unless the output is FP16
    if (out_type == GPUSQ_OUT_F16) ok = ok && make_map_y_f16(&map_y, Y, (uint64_t)M, (uint64_t)N);
    // INT8 output: box = 128 features x 32 tokens, 128-byte swizzle (the INT8 staging-tile layout)
    if (out_type == GPUSQ_OUT_I8)
        ok = ok && make_map_u8(&map_y, Y, (uint64_t)M, (uint64_t)N, 128, (uint32_t)kChunkT, CU_TENSOR_MAP_SWIZZLE_128B);
    if (!ok) return GPUSQ_ERR_CUDA;

    // launches without a twin column run the instantiation that has no trace of it
    const int smem = C::kSmemBytes;
    if (out_type == GPUSQ_OUT_F16 && y_absmax && kSparse)
        return twin_col ? launch_on(gemm_i8_kernel<true, GPUSQ_OUT_F16, false, true, true>, C::kThreads, smem, map_a, map_b, map_b2, map_e, map_y, p, clusters, stream)
                        : launch_on(gemm_i8_kernel<true, GPUSQ_OUT_F16, false, false, true>, C::kThreads, smem, map_a, map_b, map_b2, map_e, map_y, p, clusters, stream);
    if (out_type == GPUSQ_OUT_F16)
        return twin_col ? launch_on(gemm_i8_kernel<kSparse, GPUSQ_OUT_F16, false, true>, C::kThreads, smem, map_a, map_b, map_b2, map_e, map_y, p, clusters, stream)
                        : launch_on(gemm_i8_kernel<kSparse, GPUSQ_OUT_F16>, C::kThreads, smem, map_a, map_b, map_b2, map_e, map_y, p, clusters, stream);
    if (out_type == GPUSQ_OUT_I8)
        return twin_col ? launch_on(gemm_i8_kernel<kSparse, GPUSQ_OUT_I8, false, true>, C::kThreads, smem, map_a, map_b, map_b2, map_e, map_y, p, clusters, stream)
                        : launch_on(gemm_i8_kernel<kSparse, GPUSQ_OUT_I8>, C::kThreads, smem, map_a, map_b, map_b2, map_e, map_y, p, clusters, stream);
    return twin_col ? launch_on(gemm_i8_kernel<kSparse, GPUSQ_OUT_I32, false, true>, C::kThreads, smem, map_a, map_b, map_b2, map_e, map_y, p, clusters, stream)
                    : launch_on(gemm_i8_kernel<kSparse, GPUSQ_OUT_I32>, C::kThreads, smem, map_a, map_b, map_b2, map_e, map_y, p, clusters, stream);
}

// The FP16 2:4 sparse layer: binary16 activations as they are, FP32 accumulation, bias, optional GELU.
static int launch_gemm_f16(const void *X, const void *Wpacked, const float *bias, int act, int out_type, void *Y,
                           int64_t M, int N, int K, int32_t *status_buf, void *stream)
{
    using C = Cfg<true, true>;
    if (!X || !Wpacked || !Y) return GPUSQ_ERR_NULL;
    if ((out_type != GPUSQ_OUT_F16 && out_type != GPUSQ_OUT_F32) || act < 0 || act > 1) return GPUSQ_ERR_ARG;
    if (M <= 0 || N <= 0 || K <= 0 || K % 8 || M > 0x7FFFFFFF) return GPUSQ_ERR_SHAPE;
    if (out_type == GPUSQ_OUT_F16 && N % 8) return GPUSQ_ERR_SHAPE;
    if (!aligned(X, 16) || !aligned(Wpacked, 256) || !aligned(Y, 16)) return GPUSQ_ERR_ALIGN;
    if (int st = check_arch()) return st;
    if (!prepare_device(2)) return GPUSQ_ERR_CUDA;

    const int sms = num_sms();
    const int clusters = capped(max_clusters<true, true>(sms));
    if (clusters <= 0) return GPUSQ_ERR_CUDA;

    GemmParams p;
    p.w_scale = nullptr;            // the epilogue's scale is 1
    p.x_scale = nullptr;
    p.bias = bias;
    p.out_scale = nullptr;
    p.Y = Y;
    p.y_absmax = nullptr;
    p.status = status_buf;
    p.M = M;
    p.N = N;
    p.K = K;
    p.act = act;
    p.out_type = out_type;
    if (!set_tiling(p, M, N, 2 * K, clusters)) return GPUSQ_ERR_SHAPE;        // twice the bytes per column
    const bool twin_col = p.pair_tiles < p.num_tiles;
    const bool mixed = p.block_t >= 64;
    const int Kp = round_up(K, 128), Np = round_up(N, kPairF);

    // every tensor is described in bytes: kept values [Np, Kp] (Kp / 2 binary16 per row), activations
    // [M, 2 K], metadata blocks of 2 KB as 8 rows of 256 bytes
    CUtensorMap map_a, map_b, map_e;
    bool ok = make_map_u8(&map_a, Wpacked, (uint64_t)Np, (uint64_t)Kp, 128, kBlockF, CU_TENSOR_MAP_SWIZZLE_128B);
    ok = ok && make_map_u8(&map_b, X, (uint64_t)M, (uint64_t)K * 2, 128, (uint32_t)(p.block_t / 2),
                           CU_TENSOR_MAP_SWIZZLE_128B);
    CUtensorMap map_b2 = map_b;
    if (mixed)
        ok = ok && make_map_u8(&map_b2, X, (uint64_t)M, (uint64_t)K * 2, 128, (uint32_t)(p.block_t / 2 - 16),
                               CU_TENSOR_MAP_SWIZZLE_128B);
    const uint8_t *meta = reinterpret_cast<const uint8_t *>(Wpacked) + (size_t)Np * Kp;
    ok = ok && make_map_u8(&map_e, meta, (uint64_t)(Np / 128) * (Kp / 128) * 8, 256, 256, 8,
                           CU_TENSOR_MAP_SWIZZLE_NONE);
    CUtensorMap map_y = map_b;      // placeholder unless the output is FP16
    if (out_type == GPUSQ_OUT_F16) ok = ok && make_map_y_f16(&map_y, Y, (uint64_t)M, (uint64_t)N);
    if (!ok) return GPUSQ_ERR_CUDA;

    const int smem = C::kSmemBytes;
    if (out_type == GPUSQ_OUT_F16)
        return twin_col ? launch_on(gemm_i8_kernel<true, GPUSQ_OUT_F16, true, true>, C::kThreads, smem, map_a, map_b, map_b2, map_e, map_y, p, clusters, stream)
                        : launch_on(gemm_i8_kernel<true, GPUSQ_OUT_F16, true>, C::kThreads, smem, map_a, map_b, map_b2, map_e, map_y, p, clusters, stream);
    return twin_col ? launch_on(gemm_i8_kernel<true, GPUSQ_OUT_I32, true, true>, C::kThreads, smem, map_a, map_b, map_b2, map_e, map_y, p, clusters, stream)
                    : launch_on(gemm_i8_kernel<true, GPUSQ_OUT_I32, true>, C::kThreads, smem, map_a, map_b, map_b2, map_e, map_y, p, clusters, stream);
}

}  // namespace gpusq

using namespace gpusq;

extern "C" {

int gpusq_spgemm_f16(const void *X, const void *Wpacked, const float *bias, int act, int out_type, void *Y,
                     int64_t M, int N, int K, int32_t *status_buf, void *stream)
{
    return launch_gemm_f16(X, Wpacked, bias, act, out_type, Y, M, N, K, status_buf, stream);
}

int gpusq_spgemm_i8(const int8_t *Xq, const void *Wpacked, const float *w_scale, const float *x_scale,
                    const float *bias, int act, int out_type, const float *out_scale, void *Y, int64_t M, int N,
                    int K, int32_t *status_buf, void *stream)
{
    if (Wpacked && !aligned(Wpacked, 256)) return GPUSQ_ERR_ALIGN;
    return launch_gemm<true>(Xq, Wpacked, w_scale, x_scale, bias, act, out_type, out_scale, Y, M, N, K, status_buf,
                             stream);
}

int gpusq_spgemm_i8_absmax(const int8_t *Xq, const void *Wpacked, const float *w_scale, const float *x_scale,
                           const float *bias, int act, void *Y, float *y_absmax, int64_t M, int N, int K,
                           int32_t *status_buf, void *stream)
{
    if (!y_absmax) return GPUSQ_ERR_NULL;
    if (Wpacked && !aligned(Wpacked, 256)) return GPUSQ_ERR_ALIGN;
    if (!aligned(y_absmax, 4)) return GPUSQ_ERR_ALIGN;
    return launch_gemm<true>(Xq, Wpacked, w_scale, x_scale, bias, act, GPUSQ_OUT_F16, nullptr, Y, M, N, K,
                             status_buf, stream, y_absmax);
}

int gpusq_gemm_i8_dense(const int8_t *Xq, const int8_t *Wq, const float *w_scale, const float *x_scale,
                        const float *bias, int act, int out_type, const float *out_scale, void *Y, int64_t M, int N,
                        int K, int32_t *status_buf, void *stream)
{
    return launch_gemm<false>(Xq, Wq, w_scale, x_scale, bias, act, out_type, out_scale, Y, M, N, K, status_buf,
                              stream);
}

int gpusq_set_block_tokens(int block_t)
{
    if (block_t != 0 && (block_t < 32 || block_t > kMaxBlockT || block_t % 32)) return GPUSQ_ERR_ARG;
    g_block_t_override.store(block_t, std::memory_order_relaxed);
    g_n_big_override.store(-1, std::memory_order_relaxed);
    return GPUSQ_OK;
}

int gpusq_set_gemm_wait(unsigned limit_us, int withhold_loads)
{
    if (limit_us == 0) return GPUSQ_ERR_ARG;
    g_wait_us.store(limit_us, std::memory_order_relaxed);
    g_withhold_loads.store(withhold_loads ? 1 : 0, std::memory_order_relaxed);
    return GPUSQ_OK;
}

int gpusq_set_max_clusters(int clusters)
{
    if (clusters < 0) return GPUSQ_ERR_ARG;
    g_cluster_cap.store(clusters, std::memory_order_relaxed);
    return GPUSQ_OK;
}

int gpusq_set_tile_mix(int block_t, int n_big)
{
    if (block_t < 64 || block_t > kMaxBlockT || block_t % 32 || n_big < 0) return GPUSQ_ERR_ARG;
    g_block_t_override.store(block_t, std::memory_order_relaxed);
    g_n_big_override.store(n_big, std::memory_order_relaxed);
    return GPUSQ_OK;
}

}  // extern "C"
