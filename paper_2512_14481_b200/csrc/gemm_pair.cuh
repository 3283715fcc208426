// CTA-pair kernel (cta_group::2) with the activation quantizer inside, for one or several problems per launch.
#pragma once

#include "linear_common.cuh"

namespace sasq {
namespace {

// ---------------------------------------------------------------------------
// CTA-pair kernel (cta_group::2): two CTAs on neighbouring SMs share one 256 x BN
// output tile.  CTA r of the pair keeps rows [128 r, 128 r + 128) of A and rows
// [BN/2 r, BN/2 (r+1)) of W in its own shared memory, so each byte of W is read
// from shared memory by one SM only while feeding both tensor cores; at the int8
// rate a single CTA's 128 x 256 tile needs more shared-memory bandwidth (TMA
// writes + operand reads) than one SM has.  The leader CTA (rank 0) issues the
// MMAs; completion is multicast to the barriers of both CTAs.
//
// Tiling: every 256-row block of the output is cut into the same number of
// column tiles whose widths are multiples of 16 and differ by at most 16, so
// no tile is ragged; that number is chosen per problem so that the tiles fill
// whole waves of the resident pairs (plan_pair_tiles).
//
// The tensor pipe takes the next MMA only when the one before it is nearly
// done, so whatever the issuing lane does between two MMAs is time the pipe
// idles: the issue loop runs in one elected lane with nothing in it but the
// barrier poll, two descriptor adds, the MMAs and the commit.
// ---------------------------------------------------------------------------
constexpr int PBM = 256;                 // rows per pair tile
#ifndef SASQ_PAIR_STAGES
#define SASQ_PAIR_STAGES 6       // 6 x 32 KB + 32 KB of output staging + barriers = 226 KB of the 227 KB a CTA may have
#endif
constexpr int P_STAGES = SASQ_PAIR_STAGES;
constexpr int P_A_BYTES = 128 * BK;      // per CTA: 128 rows of A
constexpr int P_B_BYTES_MAX = 128 * BK;  // per CTA: up to 128 rows of W
constexpr int P_STAGE_BYTES = P_A_BYTES + P_B_BYTES_MAX;
// A stage holds the CTA's half of the W tile first, then its rows of A.  The kernel exists in two layouts of the
// same ring: 6 stages with all 128 rows of A, and, for launches whose problems all have T <= 32, 9 stages with 32
// rows of A (only the leader CTA has rows below T and loads them; the MMA still reads 128 rows from each CTA's
// shared memory, the rest being whatever lies behind, and the accumulator rows they produce are never stored).
// Such launches stream the weights once and are bound by the weight bytes in flight: 9 x 15 KB instead of 6 x 15 KB
// per CTA.
constexpr int P_SMALL_ROWS = 32;
constexpr int P_SMALL_STAGES = (P_STAGES * P_STAGE_BYTES) / (P_B_BYTES_MAX + P_SMALL_ROWS * BK);
constexpr int P_MAX_STAGES = P_SMALL_STAGES > P_STAGES ? P_SMALL_STAGES : P_STAGES;

constexpr int P_NUM_THREADS = 448;       // 14 warps: producer, MMA issuer, 4 epilogue, 8 activation quantizer
constexpr int CONV_THREADS = 256;
constexpr int CONV_WARPS = CONV_THREADS / 32;
// 8-element items per lane and chunk = 128-bit loads in flight per lane.  A launch cannot issue an MMA before the row
// blocks of its first wave of tiles are quantized and published, and a chunk is one serial chain (load, convert,
// store, fence, publish): the chunk is sized so that the first round of chunks over all workers of the grid just
// covers those row blocks.
#ifndef SASQ_CONV_ITEMS
#define SASQ_CONV_ITEMS 10
#endif
constexpr int CONV_ITEMS = SASQ_CONV_ITEMS;
constexpr int CONV_CHUNK = 32 * CONV_ITEMS;   // items per chunk (one warp)
// The four epilogue warps of a CTA have nothing to drain until the first tile's accumulators are complete: they take
// part in the first rounds of the chunk list as workers 8..11 of their CTA.
#ifndef SASQ_PAIR_LOOK_AHEAD
#define SASQ_PAIR_LOOK_AHEAD 1
#endif
#ifndef SASQ_EPI_CONV_ROUNDS
#define SASQ_EPI_CONV_ROUNDS 1
#endif
constexpr int EPI_CONV_ROUNDS = SASQ_EPI_CONV_ROUNDS;
constexpr int CONV_HEAD_WORKERS = CONV_WARPS + 4;
constexpr int kMaxRowBlocks = 1024;      // 256-row blocks the in-kernel quantizer can publish (T <= 262144)
constexpr int kReadySlots = 32;          // concurrently running launches that can each own a set of counters

constexpr int P_OUT_BUF_BYTES = 32 * 128;        // one epilogue warp's staging tile: 32 rows x 64 columns x 2 B
constexpr int P_OUT_BYTES = 4 * 2 * P_OUT_BUF_BYTES;   // 4 warps, double buffered

struct PairTail {
    uint64_t full[P_MAX_STAGES];   // used in the leader: its producer arms it with the bytes of both CTAs' loads
    uint64_t empty[P_MAX_STAGES];  // local: MMA of the pair has consumed the stage
    uint64_t tmem_full[ACC_BUFS];  // local: accumulators of the tile are complete
    uint64_t tmem_empty[ACC_BUFS]; // used in the leader: 8 epilogue warps (4 per CTA) have drained the buffer
    float scale[256];
    float bias[256];
    uint32_t tmem_base;
    volatile int abort_flag;
    int is_last_cta;
};

// the dynamic shared memory window of a CTA without static shared memory starts 1024-byte aligned; the kernel
// checks this and reports SASQ_ERR_CUDA through the status word instead of running if it ever does not hold
constexpr size_t kPairSmemBytes = (size_t)P_STAGES * P_STAGE_BYTES + P_OUT_BYTES + sizeof(PairTail);

struct PairParams {
    LinearParams lp;
    int pair_m_blocks;  // ceil(T / 256)
    int n_tiles;        // column tiles per 256-row block
    int base_units;     // tile j is (base_units + (j < rem_units)) * 16 columns wide
    int rem_units;
    int w_box_rows;     // rows of W each CTA loads per stage: half of the widest tile
    // in-kernel activation quantizer (x == nullptr: A was quantized by an earlier launch)
    const uint16_t* x;  // [T, K] 16-bit activations
    uint8_t* a_int8;    // [T, K] int8 codes (workspace), what tmap_a reads
    unsigned* ready;    // [pair_m_blocks] 8-element items of each 256-row block that are quantized and visible; zero at launch
    unsigned* done;     // CTAs that have finished; the last one zeroes `ready` and this counter again
    float qn, qp;
    // place of this problem in a launch that runs several problems back to back
    int tile_begin;         // tiles of the problems before it
    long long chunk_begin;  // quantizer chunks of the problems before it
};

// One launch runs up to kMaxGroup independent linears back to back: every CTA pair walks one list of tiles that
// covers all of them, and the quantizer warps walk one list of chunks, so the activation quantization of a problem
// (the head of a launch) and the drain of its last tiles overlap with the MMAs of its neighbours.
constexpr int kMaxGroup = 8;
// The quantizer warps run ahead of the MMAs through the whole chunk list, so the int8 activations of every problem of
// a launch are written early and read back later: a launch takes problems only while those codes (with the weights
// streaming past them) stay in the 126 MB L2.
constexpr long long kGroupCodeBytes = 80ll << 20;
// Which tiles a pair computes.  By default pair p takes tiles p, p + pairs, ... of the launch's tile list (column
// tiles fastest, so the pairs of a wave share the rows of A and walk through W together).  When every problem has a
// single 256-row block nothing is shared between tiles, and tiles of different problems cost very different amounts
// (their K differs): the host then deals the tiles out by cost (longest first, always to the least loaded pair) and
// passes each pair's list.
constexpr int kMaxListTiles = 512;
constexpr int kMaxListPairs = 96;
struct GroupParams {
    int count;
    int num_tiles;          // over all problems
    long long num_chunks;   // quantizer chunks over all problems (0: every A was quantized by an earlier launch)
    int ready_count;        // counters the last CTA zeroes again
    unsigned* ready;
    unsigned* done;
    PairParams prob[kMaxGroup];
    int use_list;                                // 0: round-robin over the tile list; 1: the lists below
    uint16_t list_begin[kMaxListPairs + 1];      // pair p computes tile_list[list_begin[p] .. list_begin[p + 1])
    uint16_t tile_list[kMaxListTiles];
};

// the tiles of one pair, in the order it computes them
struct TileWalk {
    int at, end, step;
    bool list;
    __device__ __forceinline__ TileWalk(const GroupParams& gp, int pair_id, int num_pairs) {
        list = gp.use_list != 0;
        at = list ? (int)gp.list_begin[pair_id] : pair_id;
        end = list ? (int)gp.list_begin[pair_id + 1] : gp.num_tiles;
        step = list ? 1 : num_pairs;
    }
    __device__ __forceinline__ bool more() const { return at < end; }
    __device__ __forceinline__ void next() { at += step; }
    __device__ __forceinline__ int tile(const GroupParams& gp) const { return list ? (int)gp.tile_list[at] : at; }
    __device__ __forceinline__ bool is_last() const { return at + step >= end; }
    // tiles still to come, this one included
    __device__ __forceinline__ int remaining() const { return at < end ? (end - at + step - 1) / step : 0; }
};
// the problem tile g belongs to
__device__ __forceinline__ int problem_of(const GroupParams& gp, int g) {
    int q = 0;
    while (q + 1 < gp.count && g >= gp.prob[q + 1].tile_begin) ++q;
    return q;
}
struct GroupMaps {
    CUtensorMap a[kMaxGroup], w[kMaxGroup], y64[kMaxGroup], y16[kMaxGroup];
};

// first column and width of column tile j
__host__ __device__ __forceinline__ void pair_tile_cols(const PairParams& pp, int j, int* n0, int* width) {
    const int extra = j < pp.rem_units ? j : pp.rem_units;
    *n0 = 16 * (j * pp.base_units + extra);
    *width = 16 * (pp.base_units + (j < pp.rem_units ? 1 : 0));
}

// Eq. 1 with the fixed factor on 8 consecutive elements: one 128-bit word of 16-bit values -> 8 int8 codes.
//   t = x * fl32(1/s) (one fp32 multiply);  code = clamp(rint(t), -Qn, Qp).
// fmax first: it maps NaN to -Qn (the documented behaviour) and applies the lower clamp.  With 8 bits the upper
// clamp and the rounding are what the saturating round-to-nearest-even conversion to s32 followed by the
// saturating pack to s8 does anyway (Qn = 128, Qp = 127); narrower codes take an fmin as well.
template <bool BF, bool EIGHT_BITS>
__device__ __forceinline__ uint2 quantize8(const uint4& v, float inv, float qn, float qp) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    int c[8];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float2 f = widen2<BF>(w[q]);
        float t0 = fmaxf(__fmul_rn(f.x, inv), -qn);
        float t1 = fmaxf(__fmul_rn(f.y, inv), -qn);
        if constexpr (!EIGHT_BITS) {
            t0 = fminf(t0, qp);
            t1 = fminf(t1, qp);
        }
        c[2 * q] = __float2int_rn(t0);          // saturates at the int32 range
        c[2 * q + 1] = __float2int_rn(t1);
    }
    uint32_t lo, hi, t;
    // cvt.pack.sat.s8.s32.b32 d, a, b, c:  d = (sat8(a) << 8 | sat8(b)) | (c << 16)
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(c[3]), "r"(c[2]), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(lo) : "r"(c[1]), "r"(c[0]), "r"(t));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(c[7]), "r"(c[6]), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(c[5]), "r"(c[4]), "r"(t));
    return make_uint2(lo, hi);
}

// the same with one factor per channel: inv8 points at the reciprocals of the 8 channels of this word
template <bool BF>
__device__ __forceinline__ uint2 quantize8_channels(const uint4& v, const float* inv8, float qn, float qp) {
    const float4 ia = __ldg(reinterpret_cast<const float4*>(inv8));
    const float4 ib = __ldg(reinterpret_cast<const float4*>(inv8) + 1);
    const float inv[8] = {ia.x, ia.y, ia.z, ia.w, ib.x, ib.y, ib.z, ib.w};
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    int c[8];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float2 f = widen2<BF>(w[q]);
        c[2 * q] = __float2int_rn(fminf(fmaxf(__fmul_rn(f.x, inv[2 * q]), -qn), qp));
        c[2 * q + 1] = __float2int_rn(fminf(fmaxf(__fmul_rn(f.y, inv[2 * q + 1]), -qn), qp));
    }
    uint32_t lo, hi, t;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(c[3]), "r"(c[2]), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(lo) : "r"(c[1]), "r"(c[0]), "r"(t));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(c[7]), "r"(c[6]), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(c[5]), "r"(c[4]), "r"(t));
    return make_uint2(lo, hi);
}

__device__ __forceinline__ uint4 ld_stream16(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
// (L2 policies for this traffic were measured and not kept: storing the codes with an evict-last policy brings the
// DRAM traffic of a T = 16384 launch down from 1.23 to 1.09 times its algorithmic bytes, but the launch is not bound
// by DRAM and the sustained rate fell by 2 %; loading x with evict-first changed nothing.)

// ---- in-kernel activation quantizer: one chunk = 32 lanes x CONV_ITEMS items of 8 elements, contiguous in x ----
struct ConvJob {
    const uint4* src;            // x as 128-bit words (8 elements each)
    uint2* dst;                  // int8 codes as 64-bit words
    unsigned* ready;             // per 256-row block: items quantized and visible
    long long total;             // items in x
    long long items_per_block;   // items per 256-row block
    float inv, qn, qp;
    bool eight;
    const float* chan_inv;       // per-channel reciprocals, or NULL
    unsigned vec_per_row;        // K / 8
};

__device__ __forceinline__ void conv_load(const ConvJob& j, long long c, int lane, uint4 (&v)[CONV_ITEMS]) {
#pragma unroll
    for (int u = 0; u < CONV_ITEMS; ++u) {
        const long long i = c * CONV_CHUNK + u * 32 + lane;
        if (i < j.total) v[u] = ld_stream16(j.src + i);
    }
}

template <bool BF>
__device__ __forceinline__ void conv_store(const ConvJob& j, long long c, int lane, const uint4 (&v)[CONV_ITEMS]) {
    if (j.chan_inv != nullptr) {
#pragma unroll
        for (int u = 0; u < CONV_ITEMS; ++u) {
            const long long i = c * CONV_CHUNK + u * 32 + lane;
            if (i < j.total)
                j.dst[i] = quantize8_channels<BF>(v[u], j.chan_inv + 8 * (unsigned)(i % j.vec_per_row), j.qn, j.qp);
        }
    } else if (j.eight) {
#pragma unroll
        for (int u = 0; u < CONV_ITEMS; ++u) {
            const long long i = c * CONV_CHUNK + u * 32 + lane;
            if (i < j.total) j.dst[i] = quantize8<BF, true>(v[u], j.inv, j.qn, j.qp);
        }
    } else {
#pragma unroll
        for (int u = 0; u < CONV_ITEMS; ++u) {
            const long long i = c * CONV_CHUNK + u * 32 + lane;
            if (i < j.total) j.dst[i] = quantize8<BF, false>(v[u], j.inv, j.qn, j.qp);
        }
    }
}

// every lane's stores visible at GPU scope (and to the TMA unit), then one add per row block the chunk touches
__device__ __forceinline__ void conv_publish(const ConvJob& j, long long c, int lane) {
    asm volatile("fence.proxy.async.global;" ::: "memory");
    __syncwarp();
    if (lane == 0) {
        __threadfence();        // cumulative: orders the stores of every lane (observed through the warp barrier)
        const long long first = c * CONV_CHUNK;
        const long long end = (first + CONV_CHUNK < j.total) ? first + CONV_CHUNK : j.total;
        long long i = first;
        while (i < end) {
            const long long blk = i / j.items_per_block;
            const long long blk_end = (blk + 1) * j.items_per_block;
            const long long upto = blk_end < end ? blk_end : end;
            atomicAdd(j.ready + blk, (unsigned)(upto - i));
            i = upto;
        }
    }
}

// Bounded wait until *counter (written by other CTAs with a fence before their atomic add) reaches `need`.
__device__ __forceinline__ bool wait_rows_ready(const unsigned* counter, unsigned need, PairTail* tail,
                                                const LinearParams& p) {
    const long long t0 = clock64();
    int polls = 0;
    for (;;) {
        unsigned v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
        if (v >= need) return true;
        if (p.wait_limit <= 0 || (++polls & 15) == 0) {
            if (tail->abort_flag) return false;
            if (clock64() - t0 > p.wait_limit) {
                tail->abort_flag = 1;
                atomicMax(p.status, (int)SASQ_ERR_TIMEOUT);
                return false;
            }
        }
        __nanosleep(64);
    }
}

__device__ __forceinline__ bool wait_bounded_pair(uint64_t* bar, uint32_t parity, PairTail* tail,
                                                  const LinearParams& p) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    int polls = 0;
    while (!ptx::mbar_try_wait(bar, parity)) {
        if (p.wait_limit <= 0 || (++polls & 63) == 0) {      // a zero limit gives up at the first unsuccessful poll
            if (tail->abort_flag) return false;
            if (clock64() - t0 > p.wait_limit) {
                tail->abort_flag = 1;
                atomicMax(p.status, (int)SASQ_ERR_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}

// The chunk list of a launch (all problems, in problem order) as one worker of a CTA walks it.  Rounds below
// EPI_CONV_ROUNDS are dealt over 12 workers per CTA (the quantizer warps, slots 0..7, and the epilogue warps, slots
// 8..11), later rounds over the 8 quantizer warps; within a round the workers of the grid take consecutive chunks, so
// the row blocks become ready in the order the tiles need them.  Every warp runs its own load -> quantize -> store ->
// fence -> publish chain with CONV_ITEMS 128-bit loads in flight per lane.
template <bool BF>
__device__ __forceinline__ void conv_rounds(const GroupParams& gp, int slot, bool epilogue_warp, int lane) {
    const long long grid = (long long)gridDim.x;
    const long long head = (long long)EPI_CONV_ROUNDS * grid * CONV_HEAD_WORKERS;
    ConvJob job{};
    int q = 0, job_q = -1;
    for (int r = 0;; ++r) {
        long long c;
        if (r < EPI_CONV_ROUNDS) {
            c = ((long long)r * grid + blockIdx.x) * CONV_HEAD_WORKERS + slot;
        } else {
            if (epilogue_warp) break;
            c = head + ((long long)(r - EPI_CONV_ROUNDS) * grid + blockIdx.x) * CONV_WARPS + slot;
        }
        if (c >= gp.num_chunks) break;          // c grows with r
        while (q + 1 < gp.count && c >= gp.prob[q + 1].chunk_begin) ++q;
        if (q != job_q) {
            const PairParams& pp = gp.prob[q];
            const LinearParams& p = pp.lp;
            job.src = reinterpret_cast<const uint4*>(pp.x);
            job.dst = reinterpret_cast<uint2*>(pp.a_int8);
            job.ready = pp.ready;
            job.total = (long long)p.T * (p.K >> 3);
            job.items_per_block = (long long)PBM * (p.K >> 3);
            job.chan_inv = p.chan_inv;
            job.vec_per_row = (unsigned)(p.K >> 3);
            job.qn = pp.qn;
            job.qp = pp.qp;
            job.eight = pp.qp == 127.0f;
        }
        const long long lc = c - gp.prob[q].chunk_begin;
        uint4 v[CONV_ITEMS];
        conv_load(job, lc, lane, v);
        if (q != job_q) {       // the factor is fetched with the chunk's loads already in flight
            const LinearParams& p = gp.prob[q].lp;
            job.inv = p.chan_inv == nullptr ? __fdiv_rn(1.0f, __ldg(p.x_scale)) : 0.0f;
            job_q = q;
        }
        conv_store<BF>(job, lc, lane, v);
        conv_publish(job, lc, lane);
    }
}

// ---- epilogue of (a share of) one tile by one warp ----
// The warp owns 32 rows (one TMEM lane quadrant of its CTA).  The tile's columns are cut into units of 64 columns
// (whole 128-byte lines) and, where the width is not a multiple of 64, trailing units of 16 columns; worker w of
// `workers` warps that share the quadrant takes units w, w + workers, ...  Per unit: TMEM -> registers -> dequantise
// -> the warp's 128-byte- (32-byte-) swizzled staging tile -> one TMA store (rows >= T and columns >= N are clipped
// by the tensor map).
struct EpiTile {
    const LinearParams* p;
    const CUtensorMap* y64;
    const CUtensorMap* y16;
    uint64_t policy;
    uint32_t taddr;         // TMEM address of the quadrant's lanes, first column of the accumulator buffer
    int n0, bn, row0;
    const float* scale;     // [bn] staged s_x * s_w[n] (or s_w[n] with per-row factors)
    const float* bias;      // [bn] staged bias
};

// Dequantisation of 8 adjacent accumulators of one row into four packed 16-bit pairs.  PLAIN: one static factor per
// tensor and no bias, the hot case: convert, one multiply, narrow.  Otherwise the per-row factor and the bias are
// applied as the flags say.  The epilogue is bound by the instructions it issues (a tile has 32768 values per CTA;
// the int -> float conversions alone keep the SM's 16-lane conversion pipe busy for 2048 cycles), so the hot case
// carries none it does not need.  (Converting on the integer and FMA pipes instead -- split the value in two
// 16-bit halves, make each a float through the mantissa of a constant, join them with one fused multiply-add --
// is exact too but costs six issue slots per value: measured 1 to 2 % slower.)
template <bool BF, bool PLAIN>
__device__ __forceinline__ uint4 dequant8(const uint32_t* v, const float* s8, const float* b8, bool per_row,
                                          float s_row, bool has_bias) {
    uint32_t o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        float f0, f1;
        if constexpr (PLAIN) {
            f0 = __fmul_rn(__int2float_rn((int)v[2 * q]), s8[2 * q]);
            f1 = __fmul_rn(__int2float_rn((int)v[2 * q + 1]), s8[2 * q + 1]);
        } else {
            f0 = __fmul_rn(__int2float_rn((int)v[2 * q]), out_scale(per_row, s_row, s8[2 * q]));
            f1 = __fmul_rn(__int2float_rn((int)v[2 * q + 1]), out_scale(per_row, s_row, s8[2 * q + 1]));
            if (has_bias) {
                f0 = __fadd_rn(f0, b8[2 * q]);
                f1 = __fadd_rn(f1, b8[2 * q + 1]);
            }
        }
        o[q] = narrow2<BF>(f0, f1);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// 16 adjacent columns of the warp's 32 rows: factors (and bias) read from the staged arrays first, then two
// 16-byte pieces written to the staging tile (`piece0`, `piece0 + 1` of a row of `row_bytes` bytes, swizzled) and,
// when asked for, the raw accumulators to acc_out.
template <bool BF, bool PLAIN>
__device__ __forceinline__ void dequant16_to_stage(const uint32_t* v, const float* sc, const float* bi, bool per_row,
                                                   float s_row, bool has_bias, uint8_t* sbuf, int lane, int row_bytes,
                                                   int piece0, int32_t* acc_dst, bool acc_ok0, bool acc_ok1) {
    // the loads of a piece before its store: the compiler cannot tell the staged factors from the staging tile and
    // keeps every load behind the store before it
    const int sw = row_bytes == 128 ? (lane & 7) : ((lane >> 2) & 1);
#pragma unroll
    for (int h8 = 0; h8 < 2; ++h8) {
        float s8[8], b8[8];
        const float4 f0 = *reinterpret_cast<const float4*>(sc + 8 * h8);
        const float4 f1 = *reinterpret_cast<const float4*>(sc + 8 * h8 + 4);
        s8[0] = f0.x; s8[1] = f0.y; s8[2] = f0.z; s8[3] = f0.w; s8[4] = f1.x; s8[5] = f1.y; s8[6] = f1.z; s8[7] = f1.w;
        if constexpr (!PLAIN) {
            if (has_bias) {
                const float4 c0 = *reinterpret_cast<const float4*>(bi + 8 * h8);
                const float4 c1 = *reinterpret_cast<const float4*>(bi + 8 * h8 + 4);
                b8[0] = c0.x; b8[1] = c0.y; b8[2] = c0.z; b8[3] = c0.w;
                b8[4] = c1.x; b8[5] = c1.y; b8[6] = c1.z; b8[7] = c1.w;
            }
        }
        const uint4 o = dequant8<BF, PLAIN>(v + 8 * h8, s8, b8, per_row, s_row, has_bias);
        *reinterpret_cast<uint4*>(sbuf + lane * row_bytes + (((piece0 + h8) ^ sw) << 4)) = o;
        if (acc_dst != nullptr && (h8 == 0 ? acc_ok0 : acc_ok1)) {
            int32_t* a = acc_dst + 8 * h8;
            *reinterpret_cast<uint4*>(a) = make_uint4(v[8 * h8], v[8 * h8 + 1], v[8 * h8 + 2], v[8 * h8 + 3]);
            *reinterpret_cast<uint4*>(a + 4) = make_uint4(v[8 * h8 + 4], v[8 * h8 + 5], v[8 * h8 + 6], v[8 * h8 + 7]);
        }
    }
}

// copy_out: the staging tile is copied to global memory by the warp itself (128-bit loads from shared memory, 128-bit
// stores, eight lanes per 128-byte row) instead of by a TMA store.  A TMA store has to have read the staging tile
// before the CTA may leave (about a microsecond after it is issued, measured), which nothing hides after the last
// tile of a pair; plain stores are simply complete when the grid is.
template <bool BF>
__device__ __forceinline__ void epilogue_units(const EpiTile& t, uint8_t* my_stage, unsigned& out_flip, int lane,
                                               int worker, int workers, bool copy_out) {
    const LinearParams& p = *t.p;
    const bool per_row = p.row_scale != nullptr;
    const bool has_bias = p.bias != nullptr;
    const bool plain = !per_row && !has_bias;
    const int row = t.row0 + lane;
    const bool row_ok = row < p.T;
    const float s_row = (per_row && row_ok) ? __ldg(p.row_scale + row) : 1.0f;
    int32_t* arow = (p.acc_out && row_ok) ? p.acc_out + (size_t)row * p.N + t.n0 : nullptr;
    uint16_t* y = reinterpret_cast<uint16_t*>(p.y);
    const int n64 = t.bn >> 6;
    const int units = n64 + ((t.bn & 63) >> 4);
#pragma unroll 1
    for (int u = worker; u < units; u += workers) {
        uint8_t* sbuf = my_stage + (size_t)(out_flip & 1) * P_OUT_BUF_BYTES;
        if (lane == 0) ptx::bulk_wait_group_read<1>();      // the store that used this buffer has read it
        __syncwarp();
        if (u < n64) {
            const int c = u << 6;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t v[32];
                ptx::tmem_ld_32x32(t.taddr + (uint32_t)(c + 32 * h), v);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int g16 = 0; g16 < 32; g16 += 16) {
                    const int col = c + 32 * h + g16;               // first of these 16 columns, within the tile
                    const bool ok0 = (t.n0 + col) < p.N, ok1 = (t.n0 + col + 8) < p.N;
                    if (plain)
                        dequant16_to_stage<BF, true>(v + g16, t.scale + col, t.bias + col, false, 1.0f, false, sbuf, lane,
                                                     128, (col & 63) >> 3, arow ? arow + col : nullptr, ok0, ok1);
                    else
                        dequant16_to_stage<BF, false>(v + g16, t.scale + col, t.bias + col, per_row, s_row, has_bias,
                                                      sbuf, lane, 128, (col & 63) >> 3, arow ? arow + col : nullptr,
                                                      ok0, ok1);
                }
            }
            if (copy_out) {
                __syncwarp();
                const int piece = lane & 7;
                const int col = t.n0 + c + piece * 8;           // N is a multiple of 8: a piece is inside or outside
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = (lane >> 3) + 4 * i;
                    const uint4 w = *reinterpret_cast<const uint4*>(sbuf + r * 128 + ((piece ^ (r & 7)) << 4));
                    if (t.row0 + r < p.T && col < p.N)
                        *reinterpret_cast<uint4*>(y + (size_t)(t.row0 + r) * p.N + col) = w;
                }
            } else {
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    ptx::tma_store_2d_hint(t.y64, sbuf, t.n0 + c, t.row0, t.policy);
                    ptx::bulk_commit_group();
                }
            }
        } else {                            // 16 columns: 32-byte rows, 32-byte swizzle
            const int c = (n64 << 6) + ((u - n64) << 4);
            uint32_t v[16];
            ptx::tmem_ld_32x16(t.taddr + (uint32_t)c, v);
            ptx::tmem_ld_wait();
            const bool ok0 = (t.n0 + c) < p.N, ok1 = (t.n0 + c + 8) < p.N;
            if (plain)
                dequant16_to_stage<BF, true>(v, t.scale + c, t.bias + c, false, 1.0f, false, sbuf, lane, 32, 0,
                                             arow ? arow + c : nullptr, ok0, ok1);
            else
                dequant16_to_stage<BF, false>(v, t.scale + c, t.bias + c, per_row, s_row, has_bias, sbuf, lane, 32, 0,
                                              arow ? arow + c : nullptr, ok0, ok1);
            if (copy_out) {
                __syncwarp();
                const int piece = lane & 1;
                const int col = t.n0 + c + piece * 8;
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int r = (lane >> 1) + 16 * i;
                    const uint4 w = *reinterpret_cast<const uint4*>(sbuf + r * 32 + ((piece ^ ((r >> 2) & 1)) << 4));
                    if (t.row0 + r < p.T && col < p.N)
                        *reinterpret_cast<uint4*>(y + (size_t)(t.row0 + r) * p.N + col) = w;
                }
            } else {
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    ptx::tma_store_2d_hint(t.y16, sbuf, t.n0 + c, t.row0, t.policy);
                    ptx::bulk_commit_group();
                }
            }
        }
        if (copy_out) __syncwarp();         // the staging tile has been read before the next unit overwrites it
        ++out_flip;
    }
}

// The last tile of a pair is drained with nothing left to overlap it: the tensor pipe of the pair idles meanwhile, and
// so does every other SM that is already done.  The eight quantizer warps, long finished, share that tile's epilogue:
// each TMEM lane quadrant is served by its epilogue warp (worker 0) and the two quantizer warps whose index has the
// same value mod 4 (workers 1 and 2).  They run the very loop the epilogue warps run (one copy of the code, already
// in the instruction cache from the tiles before: a second, cold copy took longer to fetch than the work it does).
constexpr int LAST_TILE_WORKERS = 3;

template <bool BF, bool SMALL>
__global__ void __launch_bounds__(P_NUM_THREADS, 1)
w8a8_gemm_pair_kernel(const __grid_constant__ GroupMaps maps, const __grid_constant__ GroupParams gp) {
    constexpr int STAGES = SMALL ? P_SMALL_STAGES : P_STAGES;
    constexpr int A_BYTES = SMALL ? P_SMALL_ROWS * BK : P_A_BYTES;
    constexpr int STAGE_BYTES = P_B_BYTES_MAX + A_BYTES;
    static_assert(STAGES * STAGE_BYTES <= P_STAGES * P_STAGE_BYTES, "both layouts use the same ring");
    static_assert(STAGE_BYTES % 1024 == 0, "swizzled tiles start on 1024-byte boundaries");
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* tiles = smem_raw;
    uint8_t* out_stage = tiles + (size_t)P_STAGES * P_STAGE_BYTES;          // 1024-byte aligned
    PairTail* tail = reinterpret_cast<PairTail*>(out_stage + P_OUT_BYTES);
    const LinearParams& p0 = gp.prob[0].lp;         // the status word and the wait limit are the same for all problems
    if ((ptx::smem_u32(tiles) & 1023u) != 0) {      // uniform over the grid: every CTA returns before any barrier
        if (threadIdx.x == 0) atomicMax(p0.status, (int)SASQ_ERR_CUDA);
        return;
    }

    pdl_launch_dependents();

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();        // 0 = leader

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(&tail->full[s], 1);
            ptx::mbar_init(&tail->empty[s], 1);
        }
        for (int b = 0; b < ACC_BUFS; ++b) {
            ptx::mbar_init(&tail->tmem_full[b], 1);
            ptx::mbar_init(&tail->tmem_empty[b], 8);
        }
        tail->abort_flag = 0;
        ptx::mbar_init_fence();
        for (int q = 0; q < gp.count; ++q) {
            ptx::prefetch_tensormap(&maps.a[q]);
            ptx::prefetch_tensormap(&maps.w[q]);
            ptx::prefetch_tensormap(&maps.y64[q]);
            ptx::prefetch_tensormap(&maps.y16[q]);
        }
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(&tail->tmem_base, TMEM_COLS);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync_all();            // both CTAs' barriers exist before anyone signals across the pair
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = tail->tmem_base;
    // Set-up done.  From here on memory that earlier kernels of the stream may have written (x, the factors) or may
    // still be reading (y, the workspace) is used.  The producer warp waits later: the frozen weights depend on no
    // earlier kernel, so it first puts the W halves of its first stages in flight.
    if (warp != 0) pdl_wait();

    const int pair_id = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;

    if (warp == 0) {
        // ---------------- TMA producer (both CTAs) ----------------
        if (ptx::elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int ready_blk = -1, ready_q = -1;
            bool dep_waited = false;
            for (TileWalk walk(gp, pair_id, num_pairs); walk.more() && ok; walk.next()) {
                const int g = walk.tile(gp);
                const int q = problem_of(gp, g);
                const PairParams& pp = gp.prob[q];
                const LinearParams& p = pp.lp;
                const CUtensorMap* tmap_a = &maps.a[q];
                const CUtensorMap* tmap_w = &maps.w[q];
                // bytes both CTAs' loads deliver per stage: two halves of the W tile, and A from both (or, in the
                // small layout, from the leader alone)
                const uint32_t stage_tx = (uint32_t)(2 * pp.w_box_rows * BK + (SMALL ? A_BYTES : 2 * A_BYTES));
                const bool load_a = !SMALL || rank == 0;
                const int tile = g - pp.tile_begin;
                const int m_blk = tile / pp.n_tiles;
                int n0, bn;
                pair_tile_cols(pp, tile - m_blk * pp.n_tiles, &n0, &bn);
                const int a_row = m_blk * PBM + (int)rank * 128;
                // this CTA's half of the tile's W rows; the box is as high as half the widest tile, so a narrower
                // tile fetches 8 rows it does not use (rows past N read as zero)
                const int w_row = n0 + (int)rank * (bn >> 1);
                int kb_a = 0;            // k-blocks of this tile whose W half is already on its way
                if (pp.x != nullptr && (m_blk != ready_blk || q != ready_q)) {
                    // The rows of this block must have been quantized, by whichever CTAs had them, and be visible
                    // to the TMA unit before the first A load of the tile.  W does not depend on that: while
                    // waiting, fill the free stages with the W halves of the first k-blocks.
                    const int rows = p.T - m_blk * PBM;
                    const unsigned need = (unsigned)((rows < PBM ? rows : PBM) * (p.K >> 3));
                    int st = stage;
                    uint32_t ph = phase;
                    while (kb_a < p.k_blocks && kb_a < STAGES && ptx::mbar_test_wait(&tail->empty[st], ph ^ 1u)) {
                        const uint32_t full_leader = ptx::mapa_u32(ptx::smem_u32(&tail->full[st]), 0);
                        if (rank == 0) ptx::mbar_arrive_expect_tx(&tail->full[st], stage_tx);
                        ptx::tma_load_2d_pair(tiles + (size_t)st * STAGE_BYTES, tmap_w, full_leader, kb_a * BK, w_row);
                        ++kb_a;
                        if (++st == STAGES) { st = 0; ph ^= 1u; }
                    }
                    if (!dep_waited) { pdl_wait(); dep_waited = true; }
                    ok = wait_rows_ready(pp.ready + m_blk, need, tail, p);
                    if (!ok) break;
                    asm volatile("fence.proxy.async.global;" ::: "memory");
                    ready_blk = m_blk;
                    ready_q = q;
                }
                if (!dep_waited) { pdl_wait(); dep_waited = true; }       // codes written by an earlier launch
                // The check above costs a round trip to L2 and a proxy fence, and at the top of a tile the MMAs are
                // about to run out of stages: once the ring is full of this tile's loads the producer looks ahead
                // and, if the NEXT tile's row block is complete already (one load, no waiting), settles it here.
                const int look_kb = p.k_blocks - 1 < STAGES ? p.k_blocks - 1 : STAGES;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
#if SASQ_PAIR_LOOK_AHEAD
                    if (kb == look_kb) {
                        TileWalk nw = walk;
                        nw.next();
                        if (nw.more()) {
                            const int ng = nw.tile(gp);
                            const int nq = problem_of(gp, ng);
                            const PairParams& np = gp.prob[nq];
                            const int n_blk = (ng - np.tile_begin) / np.n_tiles;
                            if (np.x != nullptr && (n_blk != ready_blk || nq != ready_q)) {
                                const int rows = np.lp.T - n_blk * PBM;
                                const unsigned need = (unsigned)((rows < PBM ? rows : PBM) * (np.lp.K >> 3));
                                unsigned v;
                                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(np.ready + n_blk) : "memory");
                                if (v >= need) {
                                    asm volatile("fence.proxy.async.global;" ::: "memory");
                                    ready_blk = n_blk;
                                    ready_q = nq;
                                }
                            }
                        }
                    }
#endif
                    uint8_t* w_dst = tiles + (size_t)stage * STAGE_BYTES;
                    // Only the leader arms the barrier (with the bytes of both CTAs); the partner's copies
                    // may complete first, which merely drives the transaction count negative for a while:
                    // the phase cannot complete before the leader's arrival.
                    const uint32_t full_leader = ptx::mapa_u32(ptx::smem_u32(&tail->full[stage]), 0);
                    if (kb >= kb_a) {
                        ok = wait_bounded_pair(&tail->empty[stage], phase ^ 1u, tail, p);
                        if (!ok) break;
                        if (rank == 0) ptx::mbar_arrive_expect_tx(&tail->full[stage], stage_tx);
                        ptx::tma_load_2d_pair(w_dst, tmap_w, full_leader, kb * BK, w_row);
                    }
                    if (load_a) ptx::tma_load_2d_pair(w_dst + P_B_BYTES_MAX, tmap_a, full_leader, kb * BK, a_row);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            // after an abort, copies may still be in flight into this CTA's shared memory: their barrier lives in
            // the leader, so give them a bounded grace period (a copy takes microseconds) before the CTA may exit
            if (!ok) {
                const long long t0 = clock64();
                while (clock64() - t0 < (1LL << 22)) __nanosleep(1000);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA only) ----------------
        if (rank == 0 && ptx::elect_one()) {
            const uint64_t a_desc0 = ptx::smem_desc_k_major_sw128(ptx::smem_u32(tiles) + P_B_BYTES_MAX);
            const uint64_t b_desc0 = ptx::smem_desc_k_major_sw128(ptx::smem_u32(tiles));
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int it = 0;
            for (TileWalk walk(gp, pair_id, num_pairs); walk.more() && ok; walk.next(), ++it) {
                const int g = walk.tile(gp);
                const int q = problem_of(gp, g);
                const PairParams& pp = gp.prob[q];
                const LinearParams& p = pp.lp;
                int n0, bn;
                pair_tile_cols(pp, (g - pp.tile_begin) % pp.n_tiles, &n0, &bn);
                const uint32_t idesc = ptx::idesc_i8(PBM, bn);
                const int buf = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                ok = wait_bounded_pair(&tail->tmem_empty[buf], acc_phase ^ 1u, tail, p);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * 256);
                uint32_t accumulate = 0;            // the first MMA of a tile overwrites the accumulators
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    ok = wait_bounded_pair(&tail->full[stage], phase, tail, p);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    // 32 bytes of K per MMA inside the swizzled 128-byte row: +2 in the descriptor's address field
                    const uint64_t a_desc = a_desc0 + (uint64_t)(stage * (STAGE_BYTES >> 4));
                    const uint64_t b_desc = b_desc0 + (uint64_t)(stage * (STAGE_BYTES >> 4));
                    ptx::mma_i8_ss_pair(d_tmem, a_desc, b_desc, idesc, accumulate);
                    ptx::mma_i8_ss_pair_acc(d_tmem, a_desc + 2, b_desc + 2, idesc);
                    ptx::mma_i8_ss_pair_acc(d_tmem, a_desc + 4, b_desc + 4, idesc);
                    ptx::mma_i8_ss_pair_acc(d_tmem, a_desc + 6, b_desc + 6, idesc);
                    accumulate = 1u;
                    ptx::mma_commit_pair(&tail->empty[stage], 0x3);          // stage reusable once these MMAs are done
                    if (kb == p.k_blocks - 1) ptx::mma_commit_pair(&tail->tmem_full[buf], 0x3);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else {
        // ---------------- warps 2..5: epilogue; warps 6..13: activation quantizer (both CTAs) ----------------
        // All twelve first quantize: x is taken as a flat run of T * K / 8 items of 8 elements, cut into chunks that
        // are dealt over the workers of the grid in address order (conv_rounds; the epilogue warps, which have
        // nothing to drain until the first accumulators are complete, only take part in the first rounds).  With
        // several problems in the launch their chunks form one list, in problem order.
        // Then the epilogue warps drain every tile of the pair, overlapped with the MMAs of the next one, and the
        // quantizer warps join them for the last tile.
        const bool helper = warp >= 6;
        const int cw = warp - (P_NUM_THREADS - CONV_THREADS) / 32;          // 0..7 for the quantizer warps
        const int quad = warp & 3;                                           // TMEM lane quadrant of this warp
        const int et = threadIdx.x - 64;                                     // 0..127 for the epilogue warps
        if (!helper && blockIdx.x == 0 && et < gp.count) {          // one thread per problem checks its static factor
            const LinearParams& pe = gp.prob[et].lp;
            if (pe.row_scale == nullptr && pe.chan_inv == nullptr && scale_is_bad(__ldg(pe.x_scale)))
                atomicMax(pe.status, (int)SASQ_ERR_BAD_SCALE);
        }
        if (gp.num_chunks != 0) conv_rounds<BF>(gp, helper ? cw : CONV_WARPS + (warp - 2), !helper, lane);

        // The outputs are not read again by this launch: their lines should leave L2 first, during the launch (whose
        // DRAM interface is mostly idle), instead of staying behind dirty and being written back under the next kernel.
        const uint64_t y_policy = ptx::l2_policy_evict_first();
        const int worker = helper ? 1 + (cw >> 2) : 0;
        // staging tiles for the TMA stores: the epilogue warps have their own; the quantizer warps, which only work
        // on the last tile, take the first pipeline stages (the accumulators of the last tile are complete by then,
        // so every MMA of the pair has read its operands and no load is in flight)
        uint8_t* my_stage = helper ? tiles + (size_t)cw * (2 * P_OUT_BUF_BYTES)
                                   : out_stage + (size_t)quad * (2 * P_OUT_BUF_BYTES);
        bool ok = true;
        int it = 0;
        unsigned out_flip = 0;
        bool helpers_released = false;
        TileWalk walk(gp, pair_id, num_pairs);
        const bool any_tile = walk.more();
        for (; walk.more() && ok; walk.next(), ++it) {
            const bool last = walk.is_last();
            if (helper && !last) continue;
            const int g = walk.tile(gp);
            const int q = problem_of(gp, g);
            const PairParams& pp = gp.prob[q];
            const LinearParams& p = pp.lp;
            const int tile = g - pp.tile_begin;
            const int m_blk = tile / pp.n_tiles;
            EpiTile t;
            pair_tile_cols(pp, tile - m_blk * pp.n_tiles, &t.n0, &t.bn);
            const int buf = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
            if (!helper) {
                const bool one_factor = p.row_scale == nullptr && p.chan_inv == nullptr;   // one factor for the tensor
                const float sx = one_factor ? __ldg(p.x_scale) : 1.0f;
                const bool has_bias = p.bias != nullptr;
                asm volatile("bar.sync 1, 128;" ::: "memory");
                for (int j = et; j < t.bn; j += EPI_THREADS) {
                    const int n = t.n0 + j;
                    tail->scale[j] = (n < p.N) ? __fmul_rn(sx, __ldg(p.w_scale + n)) : 0.0f;
                    if (has_bias)
                        tail->bias[j] =
                            (n < p.N) ? widen1<BF>(__ldg(reinterpret_cast<const uint16_t*>(p.bias) + n)) : 0.0f;
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (last) {         // the factors of the last tile are staged: the quantizer warps may read them
                    asm volatile("bar.arrive 3, 384;" ::: "memory");
                    helpers_released = true;
                }
            } else {
                // the epilogue warps arrive here once they have staged the last tile's factors (or have given up)
                asm volatile("bar.sync 3, 384;" ::: "memory");
                ok = tail->abort_flag == 0;
            }
            if (ok) ok = wait_bounded_pair(&tail->tmem_full[buf], acc_phase, tail, p);
            if (!helper) ok = epilogue_all_ok(ok);
            if (!ok) break;
            ptx::tc_fence_after_sync();

            t.p = &p;
            t.y64 = &maps.y64[q];
            t.y16 = &maps.y16[q];
            t.policy = y_policy;
            t.taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * 256);
            t.row0 = m_blk * PBM + (int)rank * 128 + quad * 32;
            t.scale = tail->scale;
            t.bias = tail->bias;
            epilogue_units<BF>(t, my_stage, out_flip, lane, worker, last ? LAST_TILE_WORKERS : 1, last);
            ptx::tc_fence_before_sync();
            if (!helper && !last) {
                // this warp has drained the accumulator buffer: tell the leader's MMA issuer (after the last tile
                // nobody waits for it any more, and the arrival's release would wait for the copy-out stores)
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(ptx::mapa_u32(ptx::smem_u32(&tail->tmem_empty[buf]), 0));
            }
        }
        // a pair that gave up before its last tile still has its quantizer warps waiting for the hand-over
        if (!helper && any_tile && !helpers_released) asm volatile("bar.arrive 3, 384;" ::: "memory");
        // the output stores have read their shared-memory source; the writes themselves are complete by the end of
        // the grid, which is all that a later kernel or the host can observe
        if (lane == 0) ptx::bulk_wait_group_read<0>();
    }

    // ---------------- teardown ----------------
    // Neither CTA may leave while its partner can still read its shared memory, signal its barriers or
    // run MMAs into its TMEM.  The epilogues of both CTAs have seen the last tile's accumulators complete
    // (or every role has given up after a bounded wait), so a pair-wide barrier is enough.
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync_all();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
    if (gp.done != nullptr) {
        // the CTA that finishes last leaves the counters at zero for the next launch that draws them
        if (threadIdx.x == 0) tail->is_last_cta = (atomicAdd(gp.done, 1u) == gridDim.x - 1) ? 1 : 0;
        __syncthreads();
        if (tail->is_last_cta) {
            for (int i = threadIdx.x; i < gp.ready_count; i += P_NUM_THREADS) gp.ready[i] = 0u;
            if (threadIdx.x == 0) *gp.done = 0u;
        }
    }
}

}  // namespace
}  // namespace sasq
